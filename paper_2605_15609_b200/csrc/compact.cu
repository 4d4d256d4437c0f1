// Row compaction for the verification batch (Sec. 3.2 Stage 3 scores "each masked position" of each
// draft): the rows of slots that are already committed in their draft need no LM-head pass.  One
// kernel lists the masked rows in order, one copies their hidden states into a dense buffer that the
// fused kernel then reads; results are merged back to the rows' own places by the step tail.
#include "psd_internal.cuh"

namespace psd {
namespace {

// One thread block walks flags[0..n) in chunks of blockDim.x and writes, in row order, the rows whose
// flag is non-zero: row_ids[q] = row, pos[row] = q (or -1), *count = how many.
__global__ void __launch_bounds__(1024) list_rows_kernel(const int32_t* __restrict__ flags, int n,
                                                          int32_t* __restrict__ row_ids, int32_t* __restrict__ pos,
                                                          int32_t* __restrict__ count) {
    __shared__ int s_warp[32];
    __shared__ int s_base;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
    if (threadIdx.x == 0) s_base = 0;
    __syncthreads();
    for (int c0 = 0; c0 < n; c0 += blockDim.x) {
        const int r = c0 + threadIdx.x;
        const bool f = r < n && flags[r] != 0;
        const unsigned bal = __ballot_sync(0xffffffffu, f);
        if (lane == 0) s_warp[warp] = __popc(bal);
        __syncthreads();
        int before = s_base;
        for (int w = 0; w < warp; ++w) before += s_warp[w];
        const int q = before + __popc(bal & ((1u << lane) - 1u));
        if (r < n) pos[r] = f ? q : -1;
        if (f) row_ids[q] = r;
        __syncthreads();
        if (threadIdx.x == 0) {
            int tot = 0;
            for (int w = 0; w < n_warps; ++w) tot += s_warp[w];
            s_base += tot;
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) *count = s_base;
}

// dst[q, :] = src[row_ids[q], :] for q < count (count read from the device when count_dev is given).
__global__ void gather_rows_kernel(const uint4* __restrict__ src, const int32_t* __restrict__ row_ids,
                                   const int32_t* __restrict__ count_dev, int count_host, int H8,
                                   uint4* __restrict__ dst) {
    const int count = count_dev ? *count_dev : count_host;
    for (int q = blockIdx.x; q < count; q += gridDim.x) {
        const size_t s = (size_t)row_ids[q] * H8, d = (size_t)q * H8;
        for (int j = threadIdx.x; j < H8; j += blockDim.x) dst[d + j] = src[s + j];
    }
}

}  // namespace

int launch_list_rows(const int32_t* flags, int n, int32_t* row_ids, int32_t* pos, int32_t* count, cudaStream_t st) {
    list_rows_kernel<<<1, 1024, 0, st>>>(flags, n, row_ids, pos, count);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? PSD_OK : PSD_ERR_CUDA;
}

int launch_gather_rows(const void* src, const int32_t* row_ids, const int32_t* count_dev, int count_host, int max_rows,
                       int H, void* dst, cudaStream_t st) {
    int grid = max_rows < 4096 ? max_rows : 4096;
    if (grid < 1) grid = 1;
    gather_rows_kernel<<<grid, 128, 0, st>>>(reinterpret_cast<const uint4*>(src), row_ids, count_dev, count_host,
                                             H / 8, reinterpret_cast<uint4*>(dst));
    count_launch();
    return cudaGetLastError() == cudaSuccess ? PSD_OK : PSD_ERR_CUDA;
}

}  // namespace psd
