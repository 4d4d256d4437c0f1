// Split-vocabulary combine: merges the per-split (max, sum-exp, argmax) triples of every row into
// the prediction x^ = argmax_v p(v) and its confidence c = max_v p(v) = 1 / sum_v exp(l_v - max)
// (Sec. 3.1).  The merge is the usual associative one for (max, sum-exp); equal maxima keep the
// lower vocabulary index.  The order of merging is fixed, so results are bitwise reproducible.
#include "psd_internal.cuh"

namespace psd {
namespace {

struct Triple {
    float m, s;
    int32_t a;
};

__device__ __forceinline__ void merge(Triple& x, float m, float s, int32_t a) {
    if (m > x.m) {
        x.s = x.s * expf(x.m - m) + s;
        x.m = m;
        x.a = a;
    } else if (m == x.m) {
        x.s += s;
        x.a = min(x.a, a);
    } else {
        x.s += s * expf(m - x.m);   // also the NaN path: the sum becomes NaN and stays NaN
    }
}

constexpr int kRowsPerBlock = 32;
constexpr int kLanes = 8;

// Partials are stored [n_split][n_rows]; thread (lane, row) walks splits lane, lane+8, ... so that
// a warp reads 32 consecutive rows of one split (coalesced), then the 8 lanes of a row are merged
// in lane order through shared memory.
__global__ void __launch_bounds__(kRowsPerBlock * kLanes)
combine_kernel(const float* __restrict__ pm, const float* __restrict__ ps, const int32_t* __restrict__ pa,
               int n_split, int n_rows, int32_t* __restrict__ out_token, float* __restrict__ out_conf,
               float* __restrict__ out_lse) {
    __shared__ Triple sh[kLanes][kRowsPerBlock];
    const int tx = threadIdx.x & 31, lane = threadIdx.x >> 5;
    const int row = blockIdx.x * kRowsPerBlock + tx;
    Triple x{-INFINITY, 0.f, INT32_MAX};
    if (row < n_rows) {
        for (int j = lane; j < n_split; j += kLanes) {
            const size_t o = (size_t)j * n_rows + row;
            merge(x, pm[o], ps[o], pa[o]);
        }
    }
    sh[lane][tx] = x;
    __syncthreads();
    if (lane == 0 && row < n_rows) {
        for (int l = 1; l < kLanes; ++l) {
            const Triple y = sh[l][tx];
            if (y.a != INT32_MAX) merge(x, y.m, y.s, y.a);
        }
        out_token[row] = x.a;
        out_conf[row] = 1.0f / x.s;
        if (out_lse) out_lse[row] = x.m + logf(x.s);
    }
}

}  // namespace

int launch_combine(Partials part, int n_split, int n_rows, int32_t* out_token, float* out_conf,
                   float* out_lse, cudaStream_t st) {
    const int grid = (n_rows + kRowsPerBlock - 1) / kRowsPerBlock;
    combine_kernel<<<grid, kRowsPerBlock * kLanes, 0, st>>>(part.m, part.s, part.a, n_split, n_rows,
                                                           out_token, out_conf, out_lse);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? PSD_OK : PSD_ERR_CUDA;
}

}  // namespace psd
