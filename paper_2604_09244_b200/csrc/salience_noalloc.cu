// mvla_salience_noalloc: the salience scores without a context and without any allocation.
//
// Who needs this: code that must not allocate device memory when it calls in -- a serving loop whose
// memory pool was sized and frozen at start-up, a plug-in running inside another framework's
// allocator-controlled region, a real-time control thread where a cudaMalloc (which can take
// milliseconds and synchronises the device) would break the deadline.  mvla_prune_create allocates
// its workspace with cudaMalloc, so those callers cannot even build a context.  Here the only
// scratch the salience kernel needs (the per-head partial scores) lives in a fixed array inside the
// library image, and a timeout flag beside it.
//
// Consequences of a fixed array, which callers must know:
//   * it has a hard capacity (kScratchFloats); larger problems are refused with MVLA_ERR_CAPACITY;
//   * every GPU that loads the library carries the array until the process exits;
//   * all calls on one device share it, and it keeps whatever the previous call left there.  The
//     kernels overwrite every entry they later read, and the timeout flag is cleared at the start of
//     each call, so stale contents are never consumed;
//   * two calls whose GPU work can overlap (different streams, no ordering between them) race on it.
#include "common.cuh"

#include <cudaTypedefs.h>

#include <algorithm>
#include <cstring>
#include <mutex>

namespace {

constexpr int64_t kScratchFloats = 131072;       // 512 KiB: e.g. 32 heads x 4096 visual tokens
constexpr int kMaxDevices = 64;
constexpr int kMaxBatch = 64;

static __device__ __align__(256) float g_part_scratch[kScratchFloats];
static __device__ __align__(256) int g_timeout_flag[64];      // [0] is used; padded to its own 256 bytes

// Device addresses of the arrays above, looked up once per device.  In host code the names
// g_part_scratch / g_timeout_flag are only handles for the runtime, never addresses a kernel may use.
struct DeviceScratch {
    float* part;
    int* flag;
    bool ready;
};
DeviceScratch g_dev[kMaxDevices] = {};
std::mutex g_dev_mutex;          // host threads may make their first call on a device at the same time

cudaError_t scratch_for_current_device(int dev, DeviceScratch** out)
{
    std::lock_guard<std::mutex> lock(g_dev_mutex);
    DeviceScratch& d = g_dev[dev];
    if (!d.ready) {
        void *p = nullptr, *f = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&p, g_part_scratch);
        if (e != cudaSuccess) return e;
        e = cudaGetSymbolAddress(&f, g_timeout_flag);
        if (e != cudaSuccess) return e;
        d.part = static_cast<float*>(p);
        d.flag = static_cast<int*>(f);
        d.ready = true;
    }
    *out = &d;
    return cudaSuccess;
}

// attn[j] = sum over heads of the partial scores, in head order.  Device code may name the arrays
// directly.  If a bounded wait of the salience kernel gave up, the scores are poisoned with NaN so
// that the failure cannot pass unnoticed (there is no context to carry a sticky status).
__global__ void head_reduce_static_kernel(int64_t part_stride, int n_heads, int total_vis, float* __restrict__ attn)
{
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= total_vis) return;
    float acc = 0.f;
    for (int h = 0; h < n_heads; ++h) acc += g_part_scratch[static_cast<int64_t>(h) * part_stride + j];
    attn[j] = g_timeout_flag[0] != 0 ? __int_as_float(0x7fc00000) : acc;
}

}  // namespace

extern "C" int32_t mvla_salience_noalloc(int32_t device, int32_t dtype, int32_t n_heads, int32_t head_dim,
                                         int32_t batch, const mvla_sample* samples, const void* q, const void* k,
                                         int64_t rows, float* attn_out, void* stream)
{
    using namespace mvla;
    if (!samples || !q || !k || !attn_out || batch < 1 || rows < 1 || n_heads < 1) return MVLA_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(k)) & 15u) return MVLA_ERR_INVALID_ARG;
    if (device < 0 || device >= kMaxDevices) return MVLA_ERR_INVALID_ARG;
    if (dtype != MVLA_DTYPE_BF16 && dtype != MVLA_DTYPE_FP32) return MVLA_ERR_UNSUPPORTED;
    if (head_dim != 64 && head_dim != 128) return MVLA_ERR_UNSUPPORTED;

    // descriptors and sizes (kept on the stack: no heap use either)
    if (batch > kMaxBatch) return MVLA_ERR_CAPACITY;
    SampleDev plan[kMaxBatch];
    int64_t total_vis = 0;
    for (int b = 0; b < batch; ++b) {
        const mvla_sample& s = samples[b];
        if (s.n_txt < 1 || s.n_2d < 0 || s.n_3d < 0 || s.n_2d + s.n_3d < 1 || s.seq_off < 0) return MVLA_ERR_INVALID_ARG;
        if (s.n_txt > kMaxText || s.n_2d + s.n_3d > kMaxVis) return MVLA_ERR_CAPACITY;
        const int seq = s.n_txt + s.n_2d + s.n_3d;
        const int off[3] = {s.off_txt, s.off_2d, s.off_3d}, len[3] = {s.n_txt, s.n_2d, s.n_3d};
        for (int i = 0; i < 3; ++i) {
            if (off[i] < 0 || off[i] + len[i] > seq) return MVLA_ERR_INVALID_ARG;
            for (int j = i + 1; j < 3; ++j)
                if (len[i] > 0 && len[j] > 0 && off[i] < off[j] + len[j] && off[j] < off[i] + len[i])
                    return MVLA_ERR_INVALID_ARG;
        }
        if (static_cast<int64_t>(s.seq_off) + seq > rows) return MVLA_ERR_INVALID_ARG;
        SampleDev d;
        std::memset(&d, 0, sizeof d);
        d.seq_off = s.seq_off; d.off_txt = s.off_txt; d.n_txt = s.n_txt;
        d.off_2d = s.off_2d; d.n_2d = s.n_2d; d.off_3d = s.off_3d; d.n_3d = s.n_3d;
        d.vis_off = static_cast<int32_t>(total_vis);
        total_vis += s.n_2d + s.n_3d;
        plan[b] = d;
    }
    // the one capacity that the fixed array imposes
    if (static_cast<int64_t>(n_heads) * total_vis > kScratchFloats) return MVLA_ERR_CAPACITY;

    int prev = -1;
    if (cudaGetDevice(&prev) != cudaSuccess) return MVLA_ERR_CUDA;
    if (prev != device && cudaSetDevice(device) != cudaSuccess) return MVLA_ERR_CUDA;
    int32_t rc = MVLA_OK;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    do {
        DeviceScratch* sc = nullptr;
        if (scratch_for_current_device(device, &sc) != cudaSuccess) { rc = MVLA_ERR_CUDA; break; }
        if (cudaMemsetAsync(sc->flag, 0, sizeof(int), st) != cudaSuccess) { rc = MVLA_ERR_CUDA; break; }

        const bool umma = dtype == MVLA_DTYPE_BF16;
        CUtensorMap tq, tk;
        if (umma) {      // tensor maps are plain host structures filled in by the driver: no allocation
            void* fn = nullptr;
            cudaDriverEntryPointQueryResult qres;
            if (cudaGetDriverEntryPointByVersion("cuTensorMapEncodeTiled", &fn, 12000, cudaEnableDefault, &qres) != cudaSuccess ||
                qres != cudaDriverEntryPointSuccess || !fn) { rc = MVLA_ERR_CUDA; break; }
            auto encode = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(fn);
            cuuint64_t dims[3] = {static_cast<cuuint64_t>(head_dim), static_cast<cuuint64_t>(n_heads), static_cast<cuuint64_t>(rows)};
            cuuint64_t strides[2] = {static_cast<cuuint64_t>(head_dim) * 2, static_cast<cuuint64_t>(head_dim) * n_heads * 2};
            cuuint32_t estr[3] = {1, 1, 1};
            cuuint32_t box_q[3] = {64, 1, 16}, box_k[3] = {64, 1, static_cast<cuuint32_t>(kKeyTile)};
            if (encode(&tq, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(q), dims, strides, box_q, estr,
                       CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                       CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS ||
                encode(&tk, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(k), dims, strides, box_k, estr,
                       CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                       CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) { rc = MVLA_ERR_CUDA; break; }
        }
        for (int first = 0; first < batch && rc == MVLA_OK; first += kMaxChunk) {
            BatchDesc bd;
            std::memset(&bd, 0, sizeof bd);
            bd.n = std::min(kMaxChunk, batch - first);
            int max_tiles = 1, max_txt = 1;
            for (int i = 0; i < bd.n; ++i) {
                bd.s[i] = plan[first + i];
                max_tiles = std::max(max_tiles, (bd.s[i].n_2d + kKeyTile - 1) / kKeyTile + (bd.s[i].n_3d + kKeyTile - 1) / kKeyTile);
                max_txt = std::max(max_txt, bd.s[i].n_txt);
            }
            const int tiles_per_cta = (max_tiles + kMaxCluster - 1) / kMaxCluster;
            const int cluster = (max_tiles + tiles_per_cta - 1) / tiles_per_cta;
            const int npad = (max_txt + 15) / 16 * 16;
            const cudaError_t e = launch_salience(bd, dtype, n_heads, 1, head_dim, q, k, umma ? &tq : nullptr,
                                                  umma ? &tk : nullptr, umma, tiles_per_cta, cluster, npad, sc->part,
                                                  total_vis, sc->flag, AlphaOut{nullptr, 0, 0}, st);
            if (e == cudaErrorInvalidConfiguration) rc = MVLA_ERR_UNSUPPORTED;
            else if (e != cudaSuccess) rc = MVLA_ERR_CUDA;
        }
        if (rc != MVLA_OK) break;
        head_reduce_static_kernel<<<static_cast<unsigned>((total_vis + 255) / 256), 256, 0, st>>>(
            total_vis, n_heads, static_cast<int>(total_vis), attn_out);
        if (cudaGetLastError() != cudaSuccess) rc = MVLA_ERR_CUDA;
    } while (false);
    if (prev != device) cudaSetDevice(prev);
    return rc;
}
