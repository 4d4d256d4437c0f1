// A plain CUDA-core version of the fused LM-head + confidence computation (Sec. 3.1), kept as an
// independent cross-check of the tensor-core kernel: shared-memory tiled fp32 FMA, then a
// one-thread-per-row scan of each 64-column tile that keeps the running (max, sum-exp, argmax).
// It writes the same per-split partial triples as the tensor-core kernel; speed is not a goal.
#include <cuda_bf16.h>
#include "psd_internal.cuh"

namespace psd {
namespace {

constexpr int TM = 64, TN = 64, TK = 32;

__global__ void __launch_bounds__(256)
confidence_simt_kernel(const __nv_bfloat16* __restrict__ hidden, const __nv_bfloat16* __restrict__ W,
                       int n_rows, int H, int V, int tiles_per_split,
                       float* __restrict__ pm, float* __restrict__ ps, int32_t* __restrict__ pa) {
    __shared__ float As[TM][TK + 1];
    __shared__ float Bs[TN][TK + 1];
    __shared__ float Cs[TM][TN + 1];
    const int tid = threadIdx.x, ty = tid / 16, tx = tid % 16;
    const int split = blockIdx.x, row0 = blockIdx.y * TM;
    const int n_vtiles = (V + TN - 1) / TN;
    const int t_begin = split * tiles_per_split;
    const int t_end = min(n_vtiles, t_begin + tiles_per_split);

    float run_m = -INFINITY, run_s = 0.f;
    int run_a = INT32_MAX;

    for (int t = t_begin; t < t_end; ++t) {
        const int v0 = t * TN;
        float acc[4][4];
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
            for (int c = 0; c < 4; ++c) acc[a][c] = 0.f;
        for (int k0 = 0; k0 < H; k0 += TK) {
            for (int e = tid; e < TM * TK; e += 256) {
                const int r = e / TK, k = e % TK;
                const int gr = row0 + r, gv = v0 + r;
                As[r][k] = gr < n_rows ? __bfloat162float(hidden[(size_t)gr * H + k0 + k]) : 0.f;
                Bs[r][k] = gv < V ? __bfloat162float(W[(size_t)gv * H + k0 + k]) : 0.f;
            }
            __syncthreads();
#pragma unroll 8
            for (int k = 0; k < TK; ++k) {
                float a[4], b[4];
#pragma unroll
                for (int x = 0; x < 4; ++x) { a[x] = As[ty * 4 + x][k]; b[x] = Bs[tx * 4 + x][k]; }
#pragma unroll
                for (int x = 0; x < 4; ++x)
#pragma unroll
                    for (int y = 0; y < 4; ++y) acc[x][y] = fmaf(a[x], b[y], acc[x][y]);
            }
            __syncthreads();
        }
#pragma unroll
        for (int x = 0; x < 4; ++x)
#pragma unroll
            for (int y = 0; y < 4; ++y) Cs[ty * 4 + x][tx * 4 + y] = acc[x][y];
        __syncthreads();
        if (tid < TM) {
            for (int c = 0; c < TN && v0 + c < V; ++c) {
                const float l = Cs[tid][c];
                if (l > run_m) {
                    run_s = run_s * expf(run_m - l) + 1.f;
                    run_m = l;
                    run_a = v0 + c;
                } else {
                    run_s += expf(l - run_m);   // NaN logits end here and poison the sum
                }
            }
        }
        __syncthreads();
    }
    if (tid < TM && row0 + tid < n_rows) {
        const size_t o = (size_t)split * n_rows + row0 + tid;
        pm[o] = run_m;
        ps[o] = run_s;
        pa[o] = run_a;
    }
}

}  // namespace

int launch_confidence_simt(const void* hidden, const void* w, int n_rows, int H, int V,
                           Partials part, cudaStream_t st) {
    const int n_vtiles = (V + TN - 1) / TN;
    int n_split = max_splits(V);
    if (n_split > 296) n_split = 296;
    const int tiles_per_split = (n_vtiles + n_split - 1) / n_split;
    n_split = (n_vtiles + tiles_per_split - 1) / tiles_per_split;   // no empty split
    dim3 grid(n_split, (n_rows + TM - 1) / TM);
    confidence_simt_kernel<<<grid, 256, 0, st>>>(reinterpret_cast<const __nv_bfloat16*>(hidden),
                                                 reinterpret_cast<const __nv_bfloat16*>(w), n_rows, H, V,
                                                 tiles_per_split, part.m, part.s, part.a);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? n_split : PSD_ERR_CUDA;
}

}  // namespace psd
