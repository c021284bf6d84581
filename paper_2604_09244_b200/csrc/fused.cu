// Fast salience kernel for bf16 (Sec. 3.2.1 of the paper).
//
// Same decomposition as the generic salience kernel (one cluster per (sample, head), one CTA per one or
// two tiles of 128 keys; TMA -> shared memory -> tcgen05.mma -> tensor memory), but built as one short
// dependency chain, because at ~40 KB of input per CTA the kernel is latency bound:
//   * the loads are issued before anything else; tensor-memory allocation overlaps with them;
//   * each thread reads ALL its logits from tensor memory once (one wide tcgen05.ld) and keeps them in
//     registers through max -> exp2 -> sum -> weighted sum;
//   * the per-query (max, sum) pairs travel between the CTAs of a cluster as asynchronous remote
//     shared-memory stores that credit the receiver's mbarrier when they land (st.async with
//     complete_tx): one one-way trip, no cluster-wide hardware barrier and no fence on the critical path;
//   * per-head contributions are added into one 64-bit fixed-point accumulator per token (scale 2^60):
//     integer adds commute, so the sum over heads is exact and independent of scheduling.
#include "common.cuh"
#include "device_utils.cuh"
#include "select_impl.cuh"
#include "tmem_ld.cuh"
#include "tmem_plan.h"

#include <algorithm>
#include <cstring>

namespace mvla {
namespace {

constexpr int kFastThreads = 128;

__device__ __forceinline__ float ex2_approx(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// Asynchronous 8-byte store into the shared memory of CTA `rank` (same offset as `local_addr`); on
// landing it credits 8 bytes to that CTA's mbarrier at the offset of `local_bar`: the data and its
// "ready" signal travel together, one way.
__device__ __forceinline__ void st_async_peer_f32x2(uint32_t local_addr, uint32_t local_bar, uint32_t rank, float2 v)
{
    uint32_t raddr, rbar;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(raddr) : "r"(local_addr), "r"(rank));
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(rbar) : "r"(local_bar), "r"(rank));
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v2.f32 [%0], {%1, %2}, [%3];"
                 ::"r"(raddr), "f"(v.x), "f"(v.y), "r"(rbar) : "memory");
}
// Bounded wait with acquire at cluster scope (the arrivals come from other CTAs).
__device__ __forceinline__ bool mbar_wait_cluster(uint32_t bar, uint32_t parity)
{
    const uint64_t t0 = global_ns();
    for (uint32_t it = 0; it < kSpinLimit; ++it) {
        uint32_t ok;
        asm volatile("{\n\t.reg .pred p;\n\t"
                     "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
                     "selp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
        if (ok) return true;
        if ((it & 63u) == 63u && global_ns() - t0 > 1000000000ull) break;
    }
    return false;
}

// grid = (cluster size, n_heads, samples), cluster = (cluster size, 1, 1), 128 x SPLIT threads.
// TCOL: tensor-memory columns per tile (>= padded query count); NTILE: key tiles per CTA.
// SPLIT: threads per key.  1: a thread holds all the logits of its key.  2 (fixed-point accumulators only, no
// attention copy): threads t and t + 128 hold one half of the text queries each -- the chain through max,
// exponentials, sums and weighted sum is half as long per warp, and a scheduler has two warps to alternate
// between; both halves add into the key's accumulator.
template <int TCOL, int NTILE, int SPLIT>
__global__ void __launch_bounds__(kFastThreads * SPLIT, 1)
salience_fast_kernel(const __grid_constant__ BatchDesc bd, const __grid_constant__ CUtensorMap tmap_q,
                     const __grid_constant__ CUtensorMap tmap_k, int n_heads, int kv_group, int head_dim, int esize, int npad_max,
                     float* __restrict__ part, int64_t part_stride, unsigned long long* __restrict__ acc64,
                     int* status, int free_running, const AlphaOut alpha, int32_t* __restrict__ rearm, unsigned long long* __restrict__ rearm_rec,
                     unsigned long long* __restrict__ stamps, float* __restrict__ lcache, int cache_vis, int cache_cols)
{
    constexpr int CC = TCOL * NTILE;                      // tensor-memory columns of the CTA
    constexpr int TC = TCOL / SPLIT;                      // columns (text queries) of a tile that one thread holds
    constexpr int NT = kFastThreads * SPLIT;
    static_assert(TC % 16 == 0, "a thread holds whole groups of 16 queries");
    extern __shared__ uint8_t dyn_smem_raw[];
    uint8_t* dyn_smem = dyn_smem_raw + ((1024u - (smem_u32(dyn_smem_raw) & 1023u)) & 1023u);   // swizzle atoms are 1 KB
    __shared__ float s_m[kMaxText];                       // local max per query (scaled, log2 domain), -inf replaced by 0
    __shared__ alignas(16) float s_w[kMaxText];           // final weight per query
    __shared__ float2 s_peer[kMaxCluster][kMaxText];      // (raw local max, local sum) of every CTA of the cluster
    __shared__ float2 s_loc[kMaxText];                    // this CTA's pairs, staged for the push
    __shared__ float s_wred[4][kMaxText];
    __shared__ __align__(8) uint64_t s_bar[3];
    __shared__ uint32_t s_tmem;

    const SampleDev& s = bd.s[blockIdx.z];
    const int h = blockIdx.y;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int key = tid & (kFastThreads - 1);            // key of the tile(s) this thread works on
    const int kwarp = warp & 3;                           // its warp among the four that cover the 128 keys (= tensor-memory lane quarter)
    const int c0 = (tid / kFastThreads) * TC;             // first of its text queries
    // queries padded to the MMA's N granularity for THIS sample (the launch is sized for the longest text)
    const int npad = min(npad_max, (s.n_txt + 15) & ~15);
    const uint32_t crank = cluster_ctarank();
    const uint32_t csize = gridDim.x;
    const int d = head_dim;
    const int khalves = (d * esize + 127) / 128;          // 128-byte swizzle rows (64 bf16 or 128 e4m3) per key; a last partial box is zero-filled by TMA
    const int box_elems = 128 / esize;
    const float cscale = 1.4426950408889634f * rsqrtf(static_cast<float>(d));   // log2 domain
    const int tt0 = static_cast<int>(crank) * NTILE;
    uint8_t* Ks = dyn_smem;                               // [tile][khalf][128 rows x 128 B]
    uint8_t* Qs = dyn_smem + static_cast<size_t>(NTILE) * khalves * 16384;   // [khalf][npad rows x 128 B]
    const uint32_t bar_full = smem_u32(&s_bar[0]), bar_mma = smem_u32(&s_bar[1]), bar_x = smem_u32(&s_bar[2]);

    int valid[NTILE], vis0[NTILE];
    bool from_k[NTILE];                       // the tile's logits come from K (TMA + MMA); false: from the logit cache
    bool any_live = false;
    const bool caching = lcache != nullptr && s.cache_state >= 0;
#pragma unroll
    for (int t = 0; t < NTILE; ++t) {
        const TileInfo ti = tile_info(s, tt0 + t);
        valid[t] = ti.valid;
        vis0[t] = ti.vis0;
        any_live |= ti.valid > 0;
        from_k[t] = !caching || ((s.tile_compute >> (tt0 + t)) & 1u) != 0;
    }
    // row of this thread's key in the cache: [state][head][visual index][column]
    const int64_t cache_row0 = caching ? ((static_cast<int64_t>(s.cache_state) * n_heads + h) * cache_vis) * cache_cols : 0;

    if (tid == 0) {                           // the loads go out first; everything else overlaps with them
        prefetch_tensormap(&tmap_q);
        prefetch_tensormap(&tmap_k);
        mbar_init(bar_full, 1);
        mbar_init(bar_mma, 1);
        mbar_init(bar_x, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        mbar_expect_tx(bar_x, csize * static_cast<uint32_t>(npad) * 8u);     // every CTA of the cluster sends npad pairs
        // Inputs may come from the kernel before this one -- unless the host has established (stable
        // inputs, scratch ordered by events) that nothing this kernel touches depends on it.
        if (!free_running) pdl_wait();
        if (stamps) {                         // measurement aid: when this CTA was free to start its loads
            const unsigned cta = blockIdx.x + gridDim.x * (blockIdx.y + gridDim.y * blockIdx.z);
            if (cta < kStampSlots) stamps[2 * cta] = global_ns();
        }
        int live = 0;                         // key tiles to fetch: those that exist and do not come from the cache
#pragma unroll
        for (int t = 0; t < NTILE; ++t) live += valid[t] > 0 && from_k[t];
        // (no tile to compute: nothing is fetched, both barriers below complete at once)
        mbar_expect_tx(bar_full, live > 0 ? static_cast<uint32_t>(khalves) * (npad * 128 + live * 16384) : 0u);
        for (int kh = 0; kh < khalves && live > 0; ++kh)
            for (int c = 0; c < npad / 16; ++c)
                tma_load_3d(smem_u32(Qs + kh * npad * 128 + c * 2048), &tmap_q, kh * box_elems, h,
                            s.seq_off + s.off_txt + c * 16, bar_full);
#pragma unroll
        for (int t = 0; t < NTILE; ++t) {
            if (valid[t] <= 0 || !from_k[t]) continue;
            const int row0 = tile_info(s, tt0 + t).row0;
            for (int kh = 0; kh < khalves; ++kh)
                tma_load_3d(smem_u32(Ks + (t * khalves + kh) * 16384), &tmap_k, kh * box_elems, h / kv_group, row0, bar_full);
        }
    }
    if (tid < kMaxText) s_w[tid] = 0.f;
    __syncwarp();
    cluster_arrive_release();                 // publishes this CTA's barriers; matched by the wait before the first remote store
    uint32_t tmem_cols = 32;
    while (tmem_cols < static_cast<uint32_t>(CC)) tmem_cols <<= 1;
    // blocks until the columns are free: the launcher has made sure that the CTAs resident on a multiprocessor
    // never ask for more than its 512 columns together, so no CTA waits here for one that waits for it
    if (warp == 1) tmem_alloc(smem_u32(&s_tmem), tmem_cols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = s_tmem;
    // Thread 0 is past its wait for the kernel before this one, so whatever that kernel wrote is
    // complete: the next kernel may become resident now and may read such data in its prologue.
    pdl_trigger();
    // One CTA per sample re-arms the words through which the kernel after this one hands the kept list from
    // its selecting CTA to its copying CTAs (-1: not yet known).  Their last users finished long ago.
    if (rearm && blockIdx.x == 0 && blockIdx.y == 0) {
        if (!rearm_rec) {
            for (int i = tid; i < s.n_out; i += NT) rearm[s.out_off + i] = -1;
        } else {                              // the patch-by-patch tail: its list words, and three words per patch
            for (int i = tid; i < kHandWords + s.n_txt + s.n_2d + s.n_3d; i += NT) rearm[s.cap_off + i] = -1;
            for (int i = tid; i < 3 * s.n_2d; i += NT) rearm_rec[static_cast<int64_t>(s.vis_off / 2) * 3 + i] = ~0ull;
        }
    }

    if (tid == 0) {
        bool got = mbar_wait(bar_full, 0);
        if (!got) {                           // report, then give the copies one more bounded chance to land
            *reinterpret_cast<volatile int*>(status) = MVLA_ERR_TIMEOUT;
            got = mbar_wait(bar_full, 0);
        }
        if (got) {
            tc_fence_after();
            const uint32_t idesc = idesc_by_size(esize, npad);
#pragma unroll
            for (int t = 0; t < NTILE; ++t) {
                if (valid[t] <= 0 || !from_k[t]) continue;
                for (int kb = 0; kb < khalves * 4; ++kb) {     // columns past d are zeros: they add nothing
                    const int kh = kb >> 2, kin = kb & 3;          // 4 K-steps of 16 inside a 64-wide half
                    const uint64_t a = smem_desc_sw128(smem_u32(Ks + (t * khalves + kh) * 16384) + kin * 32);
                    const uint64_t b = smem_desc_sw128(smem_u32(Qs + kh * npad * 128) + kin * 32);
                    umma_by_size(esize, tmem_base + t * TCOL, a, b, idesc, kb > 0 ? 1u : 0u);
                }
            }
        }
        umma_commit(bar_mma);                 // arrives once every MMA issued above has finished
    }
    // Only thread 0 polls the barriers; the other threads park at the block barrier below (a hardware
    // wait), so while a CTA waits for its predecessor, its loads or its MMAs it leaves the issue slots and
    // the shared-memory pipe of the multiprocessor to the CTAs that share it.
    bool ok = true;
    if (tid == 0) {
        ok = mbar_wait(bar_mma, 0);
        if (!ok) *reinterpret_cast<volatile int*>(status) = MVLA_ERR_TIMEOUT;
    }
    ok = __syncthreads_and(ok) != 0;          // block-uniform from here on (aligned instructions follow)
    tc_fence_after();

    // ---- all logits of this thread's key(s) into registers, scaled to the log2 domain, masked
    float L[NTILE * TC];                      // L[t * TC + i]: tile t, text query c0 + i
    if (any_live && ok) {
        if constexpr (SPLIT == 1) {
            tmem_ld_cols<CC>(tmem_base + (static_cast<uint32_t>(kwarp * 32) << 16), L);
        } else {
#pragma unroll
            for (int t = 0; t < NTILE; ++t) {
                float part_l[TC];
                tmem_ld_cols<TC>(tmem_base + static_cast<uint32_t>(t * TCOL + c0) + (static_cast<uint32_t>(kwarp * 32) << 16), part_l);
#pragma unroll
                for (int i = 0; i < TC; ++i) L[t * TC + i] = part_l[i];
            }
        }
    } else {
#pragma unroll
        for (int i = 0; i < NTILE * TC; ++i) L[i] = 0.f;
    }
    // Logit cache: a computed tile leaves its raw dot products for the next action step, a reused tile takes
    // the previous step's instead (128 bytes per key and head at 32 queries: half a key row, and no MMA).
    if (caching && ok) {
#pragma unroll
        for (int t = 0; t < NTILE; ++t) {
            if (key >= valid[t]) continue;
            float4* row = reinterpret_cast<float4*>(lcache + cache_row0 + static_cast<int64_t>(vis0[t] + key) * cache_cols + c0);
#pragma unroll
            for (int i = 0; i < TC / 4; ++i) {
                if (c0 + 4 * i >= npad) break;
                if (from_k[t]) {
                    row[i] = make_float4(L[t * TC + 4 * i], L[t * TC + 4 * i + 1], L[t * TC + 4 * i + 2], L[t * TC + 4 * i + 3]);
                } else {
                    const float4 v = __ldcg(row + i);
                    L[t * TC + 4 * i] = v.x; L[t * TC + 4 * i + 1] = v.y; L[t * TC + 4 * i + 2] = v.z; L[t * TC + 4 * i + 3] = v.w;
                }
            }
        }
    }
    // The registers keep the raw dot products; the scale enters with the exponent below (one FFMA).  Keys
    // past the end of a ragged tile are masked; a full tile needs no pass over the registers at all, and
    // columns past the padded query count are never looked at.
#pragma unroll
    for (int t = 0; t < NTILE; ++t) {
        if (ok && valid[t] == kKeyTile) continue;         // block-uniform
        const bool live = ok && key < valid[t];
#pragma unroll
        for (int i = 0; i < TC; ++i) L[t * TC + i] = live ? L[t * TC + i] : -CUDART_INF_F;
    }

    // ---- local maximum per query
#pragma unroll
    for (int qc = 0; qc < TC / 16; ++qc) {
        if (c0 + qc * 16 >= npad) break;
        float m[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            m[i] = L[qc * 16 + i];
#pragma unroll
            for (int t = 1; t < NTILE; ++t) m[i] = fmaxf(m[i], L[t * TC + qc * 16 + i]);
        }
        const float red = warp_reduce16<true>(m, lane);
        if ((lane & 1) == 0) s_wred[kwarp][c0 + qc * 16 + col16(lane)] = red;
    }
    __syncthreads();
    float m_raw = -CUDART_INF_F;
    if (tid < npad) {
        m_raw = fmaxf(fmaxf(s_wred[0][tid], s_wred[1][tid]), fmaxf(s_wred[2][tid], s_wred[3][tid])) * cscale;
        s_m[tid] = (m_raw == -CUDART_INF_F) ? 0.f : m_raw;
    }
    __syncthreads();

    // ---- exponentials (kept in registers) and the local denominator per query
#pragma unroll
    for (int qc = 0; qc < TC / 16; ++qc) {
        if (c0 + qc * 16 >= npad) break;
        float sum[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const float mm = s_m[c0 + qc * 16 + i];
            sum[i] = 0.f;
#pragma unroll
            for (int t = 0; t < NTILE; ++t) {
                const float e = ex2_approx(fmaf(L[t * TC + qc * 16 + i], cscale, -mm));
                L[t * TC + qc * 16 + i] = e;
                sum[i] += e;
            }
        }
        const float red = warp_reduce16<false>(sum, lane);
        if ((lane & 1) == 0) s_wred[kwarp][c0 + qc * 16 + col16(lane)] = red;
    }
    __syncthreads();

    // ---- exchange (max, sum) with the other key tiles of this (sample, head)
    if (tid < npad)
        s_loc[tid] = make_float2(m_raw, (s_wred[0][tid] + s_wred[1][tid]) + (s_wred[2][tid] + s_wred[3][tid]));
    __syncthreads();
    cluster_wait_acquire();                   // every peer is running and has initialised its barriers
    for (int p = tid; p < npad * static_cast<int>(csize); p += NT) {
        const int i = p % npad;
        const uint32_t r = static_cast<uint32_t>(p / npad);
        st_async_peer_f32x2(smem_u32(&s_peer[crank][i]), bar_x, r, s_loc[i]);
    }
    __syncwarp();
    if (tid < npad) {                         // the warps that combine the pairs wait for them; the others park below
        const bool okx = mbar_wait_cluster(bar_x, 0);
        if (!okx) *reinterpret_cast<volatile int*>(status) = MVLA_ERR_TIMEOUT;
        float gmax = -CUDART_INF_F;
        for (uint32_t r = 0; r < csize; ++r) gmax = fmaxf(gmax, s_peer[r][tid].x);
        float z = 0.f;
        for (uint32_t r = 0; r < csize; ++r) {
            const float2 pr = s_peer[r][tid];
            if (pr.x > -CUDART_INF_F) z += pr.y * ex2_approx(pr.x - gmax);
        }
        const float inv_hn = 1.f / (static_cast<float>(n_heads) * static_cast<float>(s.n_txt));
        s_w[tid] = (tid < s.n_txt && z > 0.f && okx) ? ex2_approx(s_m[tid] - gmax) / z * inv_hn : 0.f;
    }
    __syncthreads();

    // ---- per key: sum over queries of the normalised probabilities (this head's contribution)
    if (!free_running) pdl_wait();            // the accumulators were read and cleared by an earlier selection
#pragma unroll
    for (int t = 0; t < NTILE; ++t) {
        if (valid[t] <= 0) continue;
        float acc = 0.f;
#pragma unroll
        for (int qc = 0; qc < TC / 16; ++qc) {
            if (c0 + qc * 16 >= npad) break;  // columns past the padded query count were never exponentiated
#pragma unroll
            for (int i = 0; i < 16; ++i)      // s_w is 0 past the text queries
                acc = fmaf(L[t * TC + qc * 16 + i], s_w[c0 + qc * 16 + i], acc);
        }
        if (key < valid[t]) {
            if (acc64)                        // (with SPLIT = 2 both halves of the queries add into the key's accumulator)
                atomicAdd(acc64 + s.vis_off + vis0[t] + key, __float2ull_rn(acc * kFixScale));
            if constexpr (SPLIT == 1) {
                if (!acc64 && part)           // neither: the caller wants the attention copy only
                    part[static_cast<int64_t>(h) * part_stride + s.vis_off + vis0[t] + key] = acc;
                if (alpha.ptr) {              // the attention itself, for the per-patch indicators: this key's row of queries
                    float4* ap = reinterpret_cast<float4*>(alpha.ptr + static_cast<int64_t>(h) * alpha.stride_h +
                                                           static_cast<int64_t>(s.vis_off + vis0[t] + key) * alpha.stride_j);
                    const float hn = static_cast<float>(n_heads) * static_cast<float>(s.n_txt);   // s_w carries 1 / (H n_t)
#pragma unroll
                    for (int g4 = 0; g4 < TCOL / 4; ++g4) {   // 16-byte stores: a handful of instructions (s_w is 0 past the text queries)
                        if (4 * g4 >= npad || 4 * g4 >= alpha.stride_j) break;
                        const float4 w4 = *reinterpret_cast<const float4*>(&s_w[4 * g4]);
                        ap[g4] = make_float4(L[t * TCOL + 4 * g4] * w4.x * hn, L[t * TCOL + 4 * g4 + 1] * w4.y * hn,
                                             L[t * TCOL + 4 * g4 + 2] * w4.z * hn, L[t * TCOL + 4 * g4 + 3] * w4.w * hn);
                    }
                }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, tmem_cols);    // the warp that allocated
    if (stamps && tid == 0) {
        const unsigned cta = blockIdx.x + gridDim.x * (blockIdx.y + gridDim.y * blockIdx.z);
        if (cta < kStampSlots) stamps[2 * cta + 1] = global_ns();
    }
}

template <int TCOL, int NTILE, int SPLIT>
cudaError_t launch_fast_t(const BatchDesc& bd, int n_heads, int kv_group, int head_dim, int esize, const CUtensorMap* tq,
                          const CUtensorMap* tk, int cluster, int npad, float* part, int64_t part_stride,
                          unsigned long long* acc64, int* status, int free_running, AlphaOut alpha, int32_t* rearm, unsigned long long* rearm_rec, unsigned long long* stamps,
                          float* lcache, int cache_vis, int cache_cols, cudaStream_t stream)
{
    size_t smem = 1024 + static_cast<size_t>((head_dim * esize + 127) / 128) * (static_cast<size_t>(NTILE) * 16384 + npad * 128);
    auto kern = salience_fast_kernel<TCOL, NTILE, SPLIT>;
    // resident CTAs x tensor-memory columns must not exceed the 512 of a multiprocessor
    const int tmem_cols = tmem_cols_for(TCOL * NTILE);
    smem = smem_for_tmem(smem, tmem_cols);
    if (smem == 0) return cudaErrorInvalidConfiguration;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return e;
    int resident = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&resident, kern, kFastThreads * SPLIT, smem);
    if (e != cudaSuccess) return e;
    if (resident * tmem_cols > kTmemColsPerSm) return cudaErrorInvalidConfiguration;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(cluster, n_heads, bd.n);
    cfg.blockDim = dim3(kFastThreads * SPLIT);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = cluster;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1] = pdl_attribute();
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, kern, bd, *tq, *tk, n_heads, kv_group, head_dim, esize, npad, part, part_stride, acc64, status, free_running, alpha, rearm, rearm_rec, stamps, lcache, cache_vis, cache_cols);
}

}  // namespace

bool fast_salience_supported(int tiles_per_cta) { return tiles_per_cta >= 1 && tiles_per_cta <= 2; }

cudaError_t launch_salience_fast(const BatchDesc& bd, int n_heads, int kv_group, int head_dim, int esize, const CUtensorMap* tmap_q,
                                 const CUtensorMap* tmap_k, int tiles_per_cta, int cluster, int npad,
                                 float* part, int64_t part_stride, unsigned long long* acc64, int* status,
                                 bool free_running, AlphaOut alpha, int32_t* rearm, unsigned long long* rearm_rec, unsigned long long* stamps,
                                 float* lcache, int cache_vis, int cache_cols, cudaStream_t stream)
{
    const int tcol = npad <= 16 ? 16 : (npad <= 32 ? 32 : 64);
    // two threads per key where the kernel's outputs allow it (see the kernel) and a thread still holds 16 queries
    const int split = (acc64 && !alpha.ptr && tcol >= 32) ? 2 : 1;
#define MVLA_FAST(TC, NTL, SP)                                                                                  \
    if (tcol == TC && tiles_per_cta == NTL && split == SP)                                                      \
        return launch_fast_t<TC, NTL, SP>(bd, n_heads, kv_group, head_dim, esize, tmap_q, tmap_k, cluster, npad, part, part_stride, \
                                          acc64, status, free_running ? 1 : 0, alpha, rearm, rearm_rec, stamps, lcache, cache_vis, cache_cols, stream);
    MVLA_FAST(16, 1, 1) MVLA_FAST(32, 1, 1) MVLA_FAST(64, 1, 1) MVLA_FAST(16, 2, 1) MVLA_FAST(32, 2, 1) MVLA_FAST(64, 2, 1)
    MVLA_FAST(32, 1, 2) MVLA_FAST(64, 1, 2) MVLA_FAST(32, 2, 2) MVLA_FAST(64, 2, 2)
#undef MVLA_FAST
    return cudaErrorInvalidConfiguration;
}

}  // namespace mvla
