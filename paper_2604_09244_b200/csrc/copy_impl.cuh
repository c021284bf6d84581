// Row copy of the fused tails: 2 KB segments, two per warp in flight; and the bounded wait on a 4-byte
// hand-over word through which a selecting CTA tells the copying CTAs of the same kernel which row goes where.
#pragma once

#include "common.cuh"
#include "device_utils.cuh"

namespace mvla {

// Which CTA of the launch this is, in the order in which the CTAs STARTED: a ticket from a counter that counts
// 0 .. grid - 1 and wraps back to 0 with the launch's last ticket (so it needs no reset between launches; one
// launch at a time per counter).  A CTA that waits for CTAs with lower tickets waits for CTAs that are running
// -- whatever order the hardware dispatches block indices in.  Called by all threads of the CTA.
__device__ __forceinline__ int cta_ticket(unsigned int* counter)
{
    __shared__ int s_ticket;
    if (threadIdx.x == 0) s_ticket = static_cast<int>(atomicInc(counter, gridDim.x - 1));
    __syncthreads();
    return s_ticket;
}

__device__ __forceinline__ uint4 ld_row(const uint4* p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ void st_row(uint4* p, const uint4& v)
{
    asm volatile("st.global.cs.v4.u32 [%0], {%1, %2, %3, %4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

// Copies `n_rows` rows.  The work is cut into 2 KB segments of one row of one tensor; warp `w` of `nw`
// takes segments w, w + nw, ... and keeps two of them (8 x 16 bytes per lane) in flight.
// rows(i, src_row, dst_row): absolute source and destination row of the i-th row of the list; false: skip it.
template <class RowFn>
__device__ __forceinline__ void copy_rows(const CompactArgs& a, int n_rows, int w, int nw, int lane, RowFn rows)
{
    const int per_row = a.seg_begin[3];
    const int n_units = n_rows * per_row;
    for (int u0 = w; u0 < n_units; u0 += 2 * nw) {
        uint4 v[2][4];
        const uint4* sp[2];
        uint4* dp[2];
        int nvec[2];
#pragma unroll
        for (int k = 0; k < 2; ++k) {
            const int u = u0 + k * nw;
            nvec[k] = 0;
            sp[k] = nullptr;
            dp[k] = nullptr;
            if (u < n_units) {
                const int r = u / per_row, g = u - r * per_row;
                int64_t srow = 0, drow = 0;
                if (!rows(r, srow, drow)) continue;
                const int tsel = g >= a.seg_begin[2] ? 2 : (g >= a.seg_begin[1] ? 1 : 0);
                const int seg = g - a.seg_begin[tsel];
                const int rb = a.row_bytes[tsel];
                sp[k] = reinterpret_cast<const uint4*>(a.src[tsel] + srow * rb + static_cast<int64_t>(seg) * kSegBytes);
                dp[k] = reinterpret_cast<uint4*>(a.dst[tsel] + drow * rb + static_cast<int64_t>(seg) * kSegBytes);
                nvec[k] = min(kSegBytes, rb - seg * kSegBytes) >> 4;
            }
        }
#pragma unroll
        for (int k = 0; k < 2; ++k)
#pragma unroll
            for (int i = 0; i < 4; ++i)
                if (lane + i * 32 < nvec[k]) v[k][i] = ld_row(sp[k] + lane + i * 32);
#pragma unroll
        for (int k = 0; k < 2; ++k)
#pragma unroll
            for (int i = 0; i < 4; ++i)
                if (lane + i * 32 < nvec[k]) st_row(dp[k] + lane + i * 32, v[k][i]);
    }
}

// One word of the kept list as the copiers see it: a 4-byte store is indivisible, so a copier that reads a
// value >= 0 has the row it needs, with no fence, flag or barrier between the CTA that selects and the
// CTAs that copy.  The words are -1 between launches.
__device__ __forceinline__ int ld_relaxed_gpu(const int* p)
{
    int v;
    asm volatile("ld.relaxed.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// Bounded wait for one word of the kept list.  Returns the word, or -1 when `limit_ns` ran out.
__device__ __forceinline__ int poll_word(const int* p, uint64_t t0, uint64_t limit_ns)
{
    int v = ld_relaxed_gpu(p);
    for (uint32_t it = 0; v < 0 && it < kSpinLimit; ++it) {
        __nanosleep(20);
        v = ld_relaxed_gpu(p);
        if ((it & 63u) == 63u && global_ns() - t0 > limit_ns) break;
    }
    return v;
}

}  // namespace mvla
