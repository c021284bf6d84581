// Compaction (Sec. 4.4 of the paper: tokens whose mask is 1 proceed, the others are discarded):
// gathers the kept rows of hidden / K / V into the dense pruned layout.
//
// Pure data movement, HBM bound.  One warp moves one 2 KB segment of one row of one tensor: four
// 16-byte loads per lane are issued back to back (512 bytes per lane-round in flight per warp),
// then four stores.  The loads bypass L1 (read once), the stores are streaming.
#include "common.cuh"

#include <algorithm>

namespace mvla {
namespace {

constexpr int kWarpsPerBlock = 8;

__device__ __forceinline__ uint4 ld_stream(const uint4* p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ void st_stream(uint4* p, const uint4& v)
{
    asm volatile("st.global.cs.v4.u32 [%0], {%1, %2, %3, %4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

// grid.x covers chunk_rows * segs_per_row_all warp-units.
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
compact_kernel(const __grid_constant__ BatchDesc bd, const __grid_constant__ CompactArgs a, const int32_t* __restrict__ kept_idx,
               int32_t chunk_rows, int32_t chunk_row0, const int32_t* __restrict__ out_offsets,
               int32_t chunk_first, int32_t batch_total)
{
    const int lane = threadIdx.x & 31;
    const int per_row = a.seg_begin[3];
    int64_t unit = static_cast<int64_t>(blockIdx.x) * kWarpsPerBlock + (threadIdx.x >> 5);
    int64_t n_units = static_cast<int64_t>(chunk_rows) * per_row;
    if (!out_offsets && unit >= n_units) return;

    asm volatile("griddepcontrol.wait;" ::: "memory");      // kept_idx comes from the kernel before this one
    // Only now may the next kernel become resident: by then this step's selection is complete.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // Row count known only on the device: the launch covers a capacity bound with a bounded grid, and the
    // warps stride over the rows that exist.
    const int64_t stride = out_offsets ? static_cast<int64_t>(gridDim.x) * kWarpsPerBlock : n_units;
    if (out_offsets) n_units = min(n_units, static_cast<int64_t>(out_offsets[batch_total] - chunk_row0) * per_row);
    for (; unit < n_units; unit += stride) {
        const int r = static_cast<int>(unit / per_row);       // output row inside this chunk
        const int u = static_cast<int>(unit - static_cast<int64_t>(r) * per_row);
        const int orow = chunk_row0 + r;
        // which sample owns output row `orow` (samples are few: linear scan)
        int b = 0;
        if (out_offsets) {            // offsets known only on the device: scan the whole batch
            while (b + 1 < batch_total && orow >= out_offsets[b + 1]) ++b;
            b -= chunk_first;
            if (b < 0 || b >= bd.n) continue;    // row belongs to another launch's samples
        } else {
            while (b + 1 < bd.n && orow >= bd.s[b + 1].out_off) ++b;
        }
        const int64_t srow = static_cast<int64_t>(bd.s[b].seq_off) + kept_idx[orow];

        const int tsel = u >= a.seg_begin[2] ? 2 : (u >= a.seg_begin[1] ? 1 : 0);
        const int seg = u - a.seg_begin[tsel];
        const int rb = a.row_bytes[tsel];
        const uint8_t* sp = a.src[tsel] + srow * rb + static_cast<int64_t>(seg) * kSegBytes;
        uint8_t* dp = a.dst[tsel] + static_cast<int64_t>(orow) * rb + static_cast<int64_t>(seg) * kSegBytes;
        const int nbytes = min(kSegBytes, rb - seg * kSegBytes);
        const int nvec = nbytes >> 4;

        uint4 v[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int idx = lane + i * 32;
            if (idx < nvec) v[i] = ld_stream(reinterpret_cast<const uint4*>(sp) + idx);
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int idx = lane + i * 32;
            if (idx < nvec) st_stream(reinterpret_cast<uint4*>(dp) + idx, v[i]);
        }
    }
}

}  // namespace

int sm_count_of_current_device()
{
    static int cached[64] = {};              // 0: not looked up yet (written once per device with the same value)
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) n = 148;
        cached[dev] = n;
    }
    return cached[dev];
}

cudaError_t launch_compact(const BatchDesc& bd, const CompactJob& job, const int32_t* kept_idx,
                           int32_t chunk_rows, int32_t chunk_row0, const int32_t* out_offsets,
                           int32_t chunk_first, int32_t batch_total, cudaStream_t stream)
{
    const CompactArgs a = compact_args(job);
    const int total = a.seg_begin[3];
    if (total == 0 || chunk_rows <= 0) return cudaSuccess;
    const int64_t units = static_cast<int64_t>(chunk_rows) * total;
    int64_t blocks = (units + kWarpsPerBlock - 1) / kWarpsPerBlock;
    if (out_offsets)      // capacity launch: a bounded grid strides over the rows that exist
        blocks = std::min<int64_t>(blocks, static_cast<int64_t>(sm_count_of_current_device()) * 32);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(blocks));
    cfg.blockDim = dim3(kWarpsPerBlock * 32);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1] = {pdl_attribute()};
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, compact_kernel, bd, a, kept_idx, chunk_rows, chunk_row0, out_offsets, chunk_first,
                              batch_total);
}

}  // namespace mvla
