// The ranking and the clamped threshold count of the transfer policy (Sec. 3.2 Stage 1; App. B.2),
// shared by the chain kernels (policy.cu) and the draft-graph kernels (dag.cu).
#pragma once
#include "psd_internal.cuh"

namespace psd {

// Rank order of slots: confidence descending, then slot ascending; NaN after every number.
__device__ __forceinline__ bool ranks_before(float cj, int j, float ci, int i) {
    bool nj = isnan(cj), ni = isnan(ci);
    if (nj != ni) return ni;
    if (nj) return j < i;
    return cj > ci || (cj == ci && j < i);
}

// Number of flagged slots that rank before slot i.
__device__ __forceinline__ int rank_among(const float* s_conf, const int* s_flag, int M, float ci, int i) {
    int r = 0;
    for (int j = 0; j < M; ++j)
        r += (s_flag[j] && ranks_before(s_conf[j], j, ci, i)) ? 1 : 0;
    return r;
}

// |T| of the clamped threshold policy.
__device__ __forceinline__ int policy_count(int n_thr, int n_masked, const psd_policy_t& p) {
    int n = max(n_thr, p.k_min);
    if (p.k_max > 0) n = min(n, p.k_max);
    return min(n, n_masked);
}

}  // namespace psd
