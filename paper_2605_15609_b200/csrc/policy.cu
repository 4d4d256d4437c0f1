// Policy, draft and acceptance kernels of the PSD step (Sec. 3.2 Stages 1-3; Eq. (1), Eq. (2);
// Algorithm 1).  One thread block per sequence block, one thread per slot.  The work is a few KB
// of int32/fp32 per block, so the kernels are latency bound: every global access is a coalesced
// row read or write, ranking is done by counting in shared memory, and counts use the block-wide
// vote instructions.
#include "psd_internal.cuh"

namespace psd {
namespace {

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

__device__ __forceinline__ int node_of(const int32_t* node, int b, int n_nodes) {
    int nd = node ? node[b] : 0;
    return min(max(nd, 0), n_nodes - 1);
}

__global__ void select_kernel(const float* __restrict__ conf, const int32_t* __restrict__ tok,
                              const int32_t* __restrict__ node, int n_nodes,
                              int32_t* __restrict__ tokens, int32_t* __restrict__ mask, int M,
                              psd_policy_t p, int32_t* __restrict__ sel, int32_t* __restrict__ n_sel,
                              int32_t* __restrict__ sel_pos) {
    extern __shared__ unsigned char smem_raw[];
    float* s_conf = reinterpret_cast<float*>(smem_raw);
    int* s_flag = reinterpret_cast<int*>(s_conf + blockDim.x);
    const int b = blockIdx.x, i = threadIdx.x;
    const bool in = i < M;
    const size_t src = ((size_t)b * n_nodes + node_of(node, b, n_nodes)) * M;
    const size_t st = (size_t)b * M;
    const float c = in ? conf[src + i] : 0.f;
    const int mk = in ? (mask[st + i] != 0) : 0;
    s_conf[i] = c;
    s_flag[i] = mk;
    const int n_masked = __syncthreads_count(mk);
    const int n_thr = __syncthreads_count(mk && c > p.tau);
    const int n = policy_count(n_thr, n_masked, p);
    const int rank = mk ? rank_among(s_conf, s_flag, M, c, i) : M;
    const bool chosen = mk && rank < n;
    if (in) {
        sel[st + i] = chosen ? 1 : 0;
        if (i >= n) sel_pos[st + i] = -1;
    }
    if (chosen) {
        sel_pos[st + rank] = i;
        tokens[st + i] = tok[src + i];   // Eq. (1)
        mask[st + i] = 0;
    }
    if (i == 0) n_sel[b] = n;
}

__global__ void build_kernel(const float* __restrict__ conf, const int32_t* __restrict__ tok,
                             const int32_t* __restrict__ node, int n_nodes,
                             const int32_t* __restrict__ tokens, const int32_t* __restrict__ mask, int M,
                             psd_policy_t p, int32_t* __restrict__ sigma, int32_t* __restrict__ n_fill,
                             int32_t* __restrict__ draft_tokens, int32_t* __restrict__ draft_mask) {
    extern __shared__ unsigned char smem_raw[];
    float* s_conf = reinterpret_cast<float*>(smem_raw);
    int* s_flag = reinterpret_cast<int*>(s_conf + blockDim.x);
    const int b = blockIdx.x, i = threadIdx.x, D = p.depth;
    const bool in = i < M;
    const size_t src = ((size_t)b * n_nodes + node_of(node, b, n_nodes)) * M;
    const size_t st = (size_t)b * M;
    const float c = in ? conf[src + i] : 0.f;
    const int mk = in ? (mask[st + i] != 0) : 0;
    s_conf[i] = c;
    s_flag[i] = mk;
    const int m = __syncthreads_count(mk);
    const int rank = mk ? rank_among(s_conf, s_flag, M, c, i) : M;
    if (in && i >= m) sigma[st + i] = -1;
    if (mk) sigma[st + rank] = i;
    const long long s = p.stride > 0 ? p.stride : p.k_min;
    const int32_t cur = in ? tokens[st + i] : 0;
    const int32_t pred = mk ? tok[src + i] : 0;
    for (int d = 0; d < D; ++d) {
        const int n_d = (int)min((long long)m, (long long)d * s);
        if (i == 0) n_fill[(size_t)b * D + d] = n_d;
        if (in) {
            const bool fill = mk && rank < n_d;       // i in S_d
            const size_t o = ((size_t)b * D + d) * M + i;
            draft_tokens[o] = fill ? pred : cur;      // Eq. (2)
            draft_mask[o] = (mk && !fill) ? 1 : 0;
        }
    }
}

__global__ void accept_kernel(const int32_t* __restrict__ tokV, const float* __restrict__ confV,
                              const int32_t* __restrict__ sigma, const int32_t* __restrict__ n_fill,
                              const int32_t* __restrict__ draft_tokens, const int32_t* __restrict__ draft_mask,
                              int M, psd_policy_t p, int32_t* __restrict__ tokens, int32_t* __restrict__ mask,
                              int32_t* __restrict__ k_star, int32_t* __restrict__ n_spec,
                              int32_t* __restrict__ n_comm, int32_t* __restrict__ accepted) {
    extern __shared__ unsigned char smem_raw[];
    float* s_conf = reinterpret_cast<float*>(smem_raw);
    int* s_flag = reinterpret_cast<int*>(s_conf + blockDim.x);
    int* s_rank_of = s_flag + blockDim.x;
    __shared__ int s_nfill[PSD_MAX_DEPTH];
    __shared__ int s_first_fail;
    const int b = blockIdx.x, i = threadIdx.x, D = p.depth;
    const bool in = i < M;
    const size_t st = (size_t)b * M;
    const size_t blk = (size_t)b * D * M;

    s_rank_of[i] = -1;
    if (i < D) s_nfill[i] = n_fill[(size_t)b * D + i];
    if (i == 0) s_first_fail = D;
    __syncthreads();
    if (in) {
        const int sg = sigma[st + i];
        if (sg >= 0 && sg < M) s_rank_of[sg] = i;
    }
    __syncthreads();

    // The depth that speculates this slot: the first node whose prefix of sigma reaches its rank.
    const int r = in ? s_rank_of[i] : -1;
    int dd = D;
    if (r >= 0)
        for (int d = D - 1; d >= 1; --d)
            if (s_nfill[d] > r) dd = d;
    bool agree = false;
    if (dd < D) agree = tokV[blk + (size_t)(dd - 1) * M + i] == draft_tokens[blk + (size_t)dd * M + i];

    int first_fail = D;
    if (p.accept_mode != PSD_ACCEPT_AGREE_AND_POLICY) {
        if (dd < D) {
            const bool good = agree && (p.accept_mode == PSD_ACCEPT_AGREE_ONLY ||
                                        confV[blk + (size_t)(dd - 1) * M + i] > p.tau);
            if (!good) atomicMin(&s_first_fail, dd);
        }
        __syncthreads();
        first_fail = s_first_fail;
    } else {
        // Per depth: run the policy on the parent's node and require membership as well.
        for (int d = 1; d < D; ++d) {
            const size_t par = blk + (size_t)(d - 1) * M;
            const float c = in ? confV[par + i] : 0.f;
            const int mk = in ? (draft_mask[par + i] != 0) : 0;
            __syncthreads();
            s_conf[i] = c;
            s_flag[i] = mk;
            const int n_masked = __syncthreads_count(mk);
            const int n_thr = __syncthreads_count(mk && c > p.tau);
            const int n = policy_count(n_thr, n_masked, p);
            bool bad = false;
            if (dd == d) {
                const int rk = mk ? rank_among(s_conf, s_flag, M, c, i) : M;
                bad = !(agree && mk && rk < n);
            }
            if (__syncthreads_or(bad)) { first_fail = d; break; }
        }
    }

    // k*: the accepted node with the most filled slots, lowest index among equals.
    int best = 0, best_n = -1;
    for (int d = 0; d < first_fail; ++d)
        if (s_nfill[d] > best_n) { best = d; best_n = s_nfill[d]; }

    int32_t t = 0;
    int mk = 0;
    bool extra = false;
    if (in) {
        const size_t o = blk + (size_t)best * M + i;
        t = draft_tokens[o];
        mk = draft_mask[o] != 0;
        extra = mk && confV[o] > p.tau;     // the verifier's own predictions on node k* that pass the threshold
        if (extra) { t = tokV[o]; mk = 0; }
        tokens[st + i] = t;
        mask[st + i] = mk;
    }
    const int n_extra = __syncthreads_count(extra);
    if (i == 0) {
        k_star[b] = best;
        n_spec[b] = best_n;
        n_comm[b] = best_n + n_extra;
    }
    if (accepted && i < D) accepted[(size_t)b * D + i] = i < first_fail ? 1 : 0;
}

inline int block_threads(int M) { return ((M + 31) / 32) * 32; }

}  // namespace

int launch_select(const float* conf, const int32_t* tok, const int32_t* node, int n_nodes,
                  int32_t* tokens, int32_t* mask, int B, int M, psd_policy_t p,
                  int32_t* sel, int32_t* n_sel, int32_t* sel_pos, cudaStream_t st) {
    const int t = block_threads(M);
    select_kernel<<<B, t, (size_t)t * 8, st>>>(conf, tok, node, n_nodes, tokens, mask, M, p, sel, n_sel, sel_pos);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? PSD_OK : PSD_ERR_CUDA;
}

int launch_build(const float* conf, const int32_t* tok, const int32_t* node, int n_nodes,
                 const int32_t* tokens, const int32_t* mask, int B, int M, psd_policy_t p,
                 int32_t* sigma, int32_t* n_fill, int32_t* draft_tokens, int32_t* draft_mask,
                 cudaStream_t st) {
    const int t = block_threads(M);
    build_kernel<<<B, t, (size_t)t * 8, st>>>(conf, tok, node, n_nodes, tokens, mask, M, p, sigma, n_fill,
                                              draft_tokens, draft_mask);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? PSD_OK : PSD_ERR_CUDA;
}

int launch_accept(const int32_t* tokV, const float* confV, const int32_t* sigma, const int32_t* n_fill,
                  const int32_t* draft_tokens, const int32_t* draft_mask, int B, int M, psd_policy_t p,
                  int32_t* tokens, int32_t* mask, int32_t* k_star, int32_t* n_spec, int32_t* n_comm,
                  int32_t* accepted, cudaStream_t st) {
    // one thread per slot, and at least one per chain node (threads i < D load n_fill)
    const int t = block_threads(M > p.depth ? M : p.depth);
    accept_kernel<<<B, t, (size_t)t * 12, st>>>(tokV, confV, sigma, n_fill, draft_tokens, draft_mask, M, p,
                                                tokens, mask, k_star, n_spec, n_comm, accepted);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? PSD_OK : PSD_ERR_CUDA;
}

}  // namespace psd
