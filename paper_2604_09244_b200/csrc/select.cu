// Stand-alone select kernel: one CTA per sample running select_sample (see select_impl.cuh).
#include "common.cuh"
#include "select_impl.cuh"

namespace mvla {
namespace {

constexpr int kSelThreads = 512;

__global__ void __launch_bounds__(kSelThreads, 1)
select_kernel(const __grid_constant__ BatchDesc bd, const GateParams gp, const SelectIO io)
{
    __shared__ SelectSmem<kSelThreads> sm;
    select_sample<kSelThreads>(bd.s[blockIdx.x], blockIdx.x, gp, io, sm);
}

}  // namespace

cudaError_t launch_select(const BatchDesc& bd, const GateParams& gp, const SelectIO& io, cudaStream_t stream)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(bd.n);
    cfg.blockDim = dim3(kSelThreads);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1] = {pdl_attribute()};
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, select_kernel, bd, gp, io);
}

}  // namespace mvla
