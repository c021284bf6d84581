// Alg. 1 of the paper taken literally, patch by patch.  A patch p of a sample owns visual token p (2D)
// and visual token P + p (3D), P = n_2d = n_3d.
//
//   patch_indicators_kernel : the four indicators of every patch from the attention copy that the
//                             salience kernel leaves behind (Eq. 3-1, Eq. 3-4, Eq. P2D, Eq. P3D);
//   patch_select_kernel     : temporal predictor (Eqs. 8, 9), dual threshold (Sec. 4.1), 1-D K-Means and
//                             the semantic rules (Sec. 4.2), fusion (Sec. 4.4), then the output offsets
//                             over the batch and the ordered kept-position lists (Eq. 10).
// The two stages as kernels of their own (the stage entry points, and steps that overlap with their
// neighbours); the work itself is in patch_impl.cuh.
#include "patch_impl.cuh"

namespace mvla {
namespace {

constexpr int kPatchThreads = 256;

// grid = (ceil(max P / PP), samples)
template <typename T, int PP>
__global__ void __launch_bounds__(kIndThreads, 1)
patch_indicators_kernel(const __grid_constant__ BatchDesc bd, int n_heads, const AlphaOut alpha,
                        const T* __restrict__ hidden, int d_model, float* __restrict__ x_out,
                        float* __restrict__ attn_out)
{
    patch_indicators_block<T, PP>(bd.s[blockIdx.y], blockIdx.x, n_heads, alpha, hidden, d_model, x_out, attn_out, nullptr, true);
}

// grid = samples
__global__ void __launch_bounds__(kPatchThreads, 1)
patch_select_kernel(const __grid_constant__ BatchDesc bd, const PatchParams pp, const PatchIO io)
{
    __shared__ PatchSmemT<kPatchThreads> sm;
    patch_select_block<kPatchThreads>(bd.s[blockIdx.x], blockIdx.x, gridDim.x, pp, io, sm, nullptr, nullptr);
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
