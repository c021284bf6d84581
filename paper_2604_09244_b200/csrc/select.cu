// Stand-alone select kernel: one CTA per sample running select_sample (see select_impl.cuh).
//
// 512 threads for samples of up to 2048 visual tokens, with the capacity template (elements per thread) the
// smallest that holds the largest sample of the launch: steps of independent requests run beside one another,
// and a 1024-thread CTA (64 registers per thread: a whole SM's register file) would have to wait for an SM
// that the other steps' CTAs have left.  1024 threads above that.
#include "common.cuh"
#include "select_impl.cuh"

namespace mvla {
namespace {

template <int NT, int CAP>
__global__ void __launch_bounds__(NT, 1)
select_kernel(const __grid_constant__ BatchDesc bd, const GateParams gp, const SelectIO io)
{
    __shared__ SelectSmem<NT, CAP> sm;
    select_sample<NT, CAP>(bd.s[blockIdx.x], blockIdx.x, gp, io, sm);
}

}  // namespace

cudaError_t launch_select(const BatchDesc& bd, const GateParams& gp, const SelectIO& io, cudaStream_t stream)
{
    int max_vis = 0;
    for (int b = 0; b < bd.n; ++b) max_vis = max(max_vis, bd.s[b].n_2d + bd.s[b].n_3d);
    const bool wide = max_vis > 2048;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(bd.n);
    cfg.blockDim = dim3(wide ? 1024 : 512);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1] = {pdl_attribute()};
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    // few elements per thread keep the chain short: the capacity is the smallest that holds the largest sample
    if (wide) return cudaLaunchKernelEx(&cfg, select_kernel<1024, kMaxVis>, bd, gp, io);
    if (max_vis > 1024) return cudaLaunchKernelEx(&cfg, select_kernel<512, 2048>, bd, gp, io);
    return cudaLaunchKernelEx(&cfg, select_kernel<512, 1024>, bd, gp, io);
}

}  // namespace mvla
