// Split-vocabulary combine: merges the per-split (max, sum-exp, argmax) triples of every row into
// the prediction x^ = argmax_v p(v) and its confidence c = max_v p(v) = 1 / sum_v exp(l_v - max)
// (Sec. 3.1).  The merge is the usual associative one for (max, sum-exp); equal maxima keep the
// lower vocabulary index.  The order of merging is fixed, so results are bitwise reproducible.
#include "combine.cuh"

namespace psd {
namespace {

__global__ void __launch_bounds__(kCombineThreads)
combine_kernel(const float* __restrict__ pm, const float* __restrict__ ps, const int32_t* __restrict__ pa,
               const SplitPlan plan, int n_rows, int32_t* __restrict__ out_token, float* __restrict__ out_conf,
               float* __restrict__ out_lse, const int32_t* __restrict__ pos, float* __restrict__ out_max,
               int32_t arg_offset, int32_t* status_dev, size_t part_cap) {
    __shared__ Triple sh[kCombineLanes][kCombineRows];
    asm volatile("griddepcontrol.wait;" ::: "memory");   // the partials come from the kernel launched before
    combine_rows32(pm, ps, pa, plan, n_rows, blockIdx.x * kCombineRows, n_rows, threadIdx.x, sh, out_token,
                   out_conf, out_lse, pos, out_max, arg_offset, status_dev, part_cap);
}

}  // namespace

int launch_combine(Partials part, SplitPlan plan, int n_rows, int32_t* out_token, float* out_conf,
                   float* out_lse, cudaStream_t st, const int32_t* pos, float* out_max, int32_t arg_offset,
                   int32_t* status_dev) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((n_rows + kCombineRows - 1) / kCombineRows);
    cfg.blockDim = dim3(kCombineThreads);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = pdl_enabled() ? 1 : 0;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const float* pm = part.m;
    const float* ps = part.s;
    const int32_t* pa = part.a;
    cudaError_t e = cudaLaunchKernelEx(&cfg, combine_kernel, pm, ps, pa, plan, n_rows, out_token, out_conf, out_lse, pos,
                                       out_max, arg_offset, status_dev, part.cap);
    count_launch();
    return e == cudaSuccess ? PSD_OK : PSD_ERR_CUDA;
}

}  // namespace psd
