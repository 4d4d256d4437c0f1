// Device-side merge of per-split (max, sum-exp, argmax) triples, shared by the stand-alone combine
// kernel and by the fused step-tail kernel so that both produce bitwise identical results.
#pragma once
#include "psd_internal.cuh"

namespace psd {

struct Triple {
    float m, s;
    int32_t a;
};

__device__ __forceinline__ void merge_triple(Triple& x, float m, float s, int32_t a) {
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

// status word: a negative value is an error code and stays; otherwise it counts non-finite rows
__device__ __forceinline__ void count_nonfinite_row(int32_t* status_dev) {
    int32_t v = *reinterpret_cast<volatile int32_t*>(status_dev);
    while (v >= 0 && v < INT32_MAX) {
        const int32_t seen = atomicCAS(status_dev, v, v + 1);
        if (seen == v) break;
        v = seen;
    }
}

constexpr int kCombineRows = 32;   // rows handled by one group of threads
constexpr int kCombineLanes = 8;   // threads per row
constexpr int kCombineThreads = kCombineRows * kCombineLanes;

// One group of 256 threads (g = 0..255 within the group) merges the splits of rows
// row0 .. row0+31: thread (lane = g / 32, tx = g % 32) walks splits lane, lane+8, ... of row
// row0 + tx (a warp reads 32 consecutive rows of one split: coalesced), then lane 0 merges the 8
// partial results of its row in lane order.  `sh` is this group's scratch [8][32].
// Every thread of the group must call this (it synchronises the whole block twice).
__device__ __forceinline__ void combine_rows32(const float* __restrict__ pm, const float* __restrict__ ps,
                                               const int32_t* __restrict__ pa, const SplitPlan& plan, int n_rows,
                                               int row0, int row_end, int g, Triple (*sh)[kCombineRows],
                                               int32_t* __restrict__ out_token, float* __restrict__ out_conf,
                                               float* __restrict__ out_lse, const int32_t* __restrict__ pos = nullptr,
                                               float* __restrict__ out_max = nullptr, int32_t arg_offset = 0,
                                               int32_t* status_dev = nullptr, size_t part_cap = 0) {
    const int tx = g & 31, lane = g >> 5;
    const int out_row = row0 + tx;
    // with compacted rows the partials of output row r sit in column pos[r]; -1 = the row was not scored
    const int row = out_row < row_end ? (pos ? pos[out_row] : out_row) : -1;
    Triple x{-INFINITY, 0.f, INT32_MAX};
    if (row >= 0) {
        int n_split = plan.uniform;
        if (n_split <= 0) {
            const int scored = plan.n_rows_dev ? min(max(*plan.n_rows_dev, 0), plan.n_rows) : plan.n_rows;
            n_split = carried_splits(plan.G, plan.hb, (scored + plan.tile_rows - 1) / plan.tile_rows, row / plan.tile_rows);
        }
        // debug build: the last split this row reads must lie inside the arrays
        if (!PSD_DEBUG_OK(part_cap == 0 || (n_split >= 1 && (size_t)(n_split - 1) * n_rows + row < part_cap), status_dev))
            n_split = 0;
        // The merge is a dependent chain, the loads are not: fetch a batch of splits first so that their
        // latencies overlap, then merge them in the same order as a plain loop would.
        constexpr int kBatch = 8;
        int j = lane;
        for (; j + (kBatch - 1) * kCombineLanes < n_split; j += kBatch * kCombineLanes) {
            float m[kBatch], sv[kBatch];
            int32_t a[kBatch];
#pragma unroll
            for (int u = 0; u < kBatch; ++u) {
                const size_t o = (size_t)(j + u * kCombineLanes) * n_rows + row;
                m[u] = pm[o];
                sv[u] = ps[o];
                a[u] = pa[o];
            }
#pragma unroll
            for (int u = 0; u < kBatch; ++u) merge_triple(x, m[u], sv[u], a[u]);
        }
        for (; j < n_split; j += kCombineLanes) {
            const size_t o = (size_t)j * n_rows + row;
            merge_triple(x, pm[o], ps[o], pa[o]);
        }
    }
    sh[lane][tx] = x;
    __syncthreads();
    if (lane == 0 && row >= 0) {
        for (int l = 1; l < kCombineLanes; ++l) {
            const Triple y = sh[l][tx];
            if (y.a != INT32_MAX) merge_triple(x, y.m, y.s, y.a);
        }
        if (out_max) {
            // the merged triple itself (one shard of the vocabulary): max, sum-exp, argmax as a global index
            out_max[out_row] = x.m;
            out_conf[out_row] = x.s;
            out_token[out_row] = x.a + arg_offset;
        } else {
            out_token[out_row] = x.a;
            out_conf[out_row] = 1.0f / x.s;
            if (out_lse) out_lse[out_row] = x.m + logf(x.s);
        }
        // A row whose logits held a NaN or an infinity has no defined confidence: count it.
        if (status_dev && !(isfinite(x.m) && isfinite(x.s))) count_nonfinite_row(status_dev);
    }
    __syncthreads();
}

}  // namespace psd
