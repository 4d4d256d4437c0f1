// Policy, draft and acceptance kernels of the PSD step (Sec. 3.2 Stages 1-3; Eq. (1), Eq. (2);
// Algorithm 1).  One thread block per sequence block, one thread per slot.  The work is a few KB
// of int32/fp32 per block, so the kernels are latency bound: every global access is a coalesced
// row read or write, ranking is done by counting in shared memory, and counts use the block-wide
// vote instructions.
//
// Each stage is a __device__ body that works for any block size >= M (and >= D for acceptance).
// The bodies take plain (not __restrict__) pointers: in the fused kernel a later stage reads what an
// earlier stage of the same launch wrote, so no load may go through the read-only data path.
// The stand-alone kernels wrap one body each, and step_tail_kernel runs the split-V merge and the
// three bodies back to back for one sequence block, so that a whole step is two launches.
#include "combine.cuh"
#include "policy_common.cuh"

namespace psd {
namespace {

__device__ __forceinline__ int node_of(const int32_t* node, int b, int n_nodes) {
    int nd = node ? node[b] : 0;
    return min(max(nd, 0), n_nodes - 1);
}

__device__ __forceinline__ void select_body(float* s_conf, int* s_flag,
                                            const float* conf, const int32_t* tok,
                                            const int32_t* node, int n_nodes,
                                            int32_t* tokens, int32_t* mask, int M,
                                            const psd_policy_t& p, int32_t* sel,
                                            int32_t* n_sel, int32_t* sel_pos) {
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

__device__ __forceinline__ void build_body(float* s_conf, int* s_flag,
                                           const float* conf, const int32_t* tok,
                                           const int32_t* node, int n_nodes,
                                           const int32_t* tokens, const int32_t* mask,
                                           int M, const psd_policy_t& p, int32_t* sigma,
                                           int32_t* n_fill, int32_t* draft_tokens,
                                           int32_t* draft_mask) {
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

__device__ __forceinline__ void accept_body(float* s_conf, int* s_flag, int* s_rank_of, int* s_nfill,
                                            int* s_first_fail_p,
                                            const int32_t* tokV, const float* confV,
                                            const int32_t* sigma, const int32_t* n_fill,
                                            const int32_t* draft_tokens,
                                            const int32_t* draft_mask, int M, const psd_policy_t& p,
                                            int32_t* tokens, int32_t* mask,
                                            int32_t* k_star, int32_t* n_spec,
                                            int32_t* n_comm, int32_t* accepted) {
    int& s_first_fail = *s_first_fail_p;
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

// ---- stand-alone kernels: one body each -----------------------------------------------------

__global__ void select_kernel(const float* __restrict__ conf, const int32_t* __restrict__ tok,
                              const int32_t* __restrict__ node, int n_nodes,
                              int32_t* __restrict__ tokens, int32_t* __restrict__ mask, int M,
                              psd_policy_t p, int32_t* __restrict__ sel, int32_t* __restrict__ n_sel,
                              int32_t* __restrict__ sel_pos) {
    extern __shared__ unsigned char smem_raw[];
    float* s_conf = reinterpret_cast<float*>(smem_raw);
    int* s_flag = reinterpret_cast<int*>(s_conf + blockDim.x);
    select_body(s_conf, s_flag, conf, tok, node, n_nodes, tokens, mask, M, p, sel, n_sel, sel_pos);
}

__global__ void build_kernel(const float* __restrict__ conf, const int32_t* __restrict__ tok,
                             const int32_t* __restrict__ node, int n_nodes,
                             const int32_t* __restrict__ tokens, const int32_t* __restrict__ mask, int M,
                             psd_policy_t p, int32_t* __restrict__ sigma, int32_t* __restrict__ n_fill,
                             int32_t* __restrict__ draft_tokens, int32_t* __restrict__ draft_mask) {
    extern __shared__ unsigned char smem_raw[];
    float* s_conf = reinterpret_cast<float*>(smem_raw);
    int* s_flag = reinterpret_cast<int*>(s_conf + blockDim.x);
    build_body(s_conf, s_flag, conf, tok, node, n_nodes, tokens, mask, M, p, sigma, n_fill, draft_tokens,
               draft_mask);
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
    accept_body(s_conf, s_flag, s_rank_of, s_nfill, &s_first_fail, tokV, confV, sigma, n_fill, draft_tokens,
                draft_mask, M, p, tokens, mask, k_star, n_spec, n_comm, accepted);
}

// ---- fused tail of a step --------------------------------------------------------------------
// One thread block per sequence block b: merge the split-V partials of the block's D*M rows
// (writing tokV / confV), then acceptance on the drafts being verified, the policy on node k*, and
// the drafts of the next step.  The stages hand data to each other through global memory written
// and read by the same block, ordered by __syncthreads.
struct StepTailArgs {
    const float* pm;
    const float* ps;
    const int32_t* pa;
    SplitPlan plan;
    int n_rows, M;
    const int32_t* pos;   // NULL, or the column of each row's partials when rows were compacted
    psd_policy_t p;
    int32_t* tokV;
    float* confV;
    int32_t *sigma, *n_fill, *draft_tokens, *draft_mask;
    int32_t *tokens, *mask, *k_star, *n_spec, *n_comm, *sel, *n_sel, *sel_pos;
    int32_t* status_dev;   // NULL, or the status word that counts non-finite rows
    size_t part_cap;       // triples each partial array holds (debug build)
};

__global__ void step_tail_kernel(const StepTailArgs a) {
    extern __shared__ unsigned char smem_raw[];
    float* s_conf = reinterpret_cast<float*>(smem_raw);
    int* s_flag = reinterpret_cast<int*>(s_conf + blockDim.x);
    int* s_rank_of = s_flag + blockDim.x;
    __shared__ Triple sh[4][kCombineLanes][kCombineRows];
    __shared__ int s_nfill[PSD_MAX_DEPTH];
    __shared__ int s_first_fail;
    const int b = blockIdx.x, D = a.p.depth, M = a.M;

    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");   // the partials come from the kernel launched before

    // split-V merge of rows [b*D*M, (b+1)*D*M): groups of 256 threads take 32 rows at a time
    const int groups = blockDim.x / kCombineThreads;
    const int grp = threadIdx.x / kCombineThreads, g = threadIdx.x % kCombineThreads;
    const int row_begin = b * D * M, row_end = row_begin + D * M;
    const int n_chunks = (D * M + kCombineRows - 1) / kCombineRows;
    for (int c0 = 0; c0 < n_chunks; c0 += groups) {
        const int c = c0 + grp;
        // threads of a group without a chunk still take part in the barriers inside
        const int r0 = c < n_chunks ? row_begin + c * kCombineRows : row_end;
        if (grp < groups)
            combine_rows32(a.pm, a.ps, a.pa, a.plan, a.n_rows, r0, row_end, g, sh[grp], a.tokV, a.confV,
                           nullptr, a.pos, nullptr, 0, a.status_dev, a.part_cap);
    }
    __syncthreads();

    accept_body(s_conf, s_flag, s_rank_of, s_nfill, &s_first_fail, a.tokV, a.confV, a.sigma, a.n_fill,
                a.draft_tokens, a.draft_mask, M, a.p, a.tokens, a.mask, a.k_star, a.n_spec, a.n_comm, nullptr);
    __syncthreads();
    select_body(s_conf, s_flag, a.confV, a.tokV, a.k_star, D, a.tokens, a.mask, M, a.p, a.sel, a.n_sel,
                a.sel_pos);
    __syncthreads();
    build_body(s_conf, s_flag, a.confV, a.tokV, a.k_star, D, a.tokens, a.mask, M, a.p, a.sigma, a.n_fill,
               a.draft_tokens, a.draft_mask);
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

int launch_step_tail(Partials part, SplitPlan plan, int n_rows, int B, int M, psd_policy_t p,
                     int32_t* tokV, float* confV, int32_t* sigma, int32_t* n_fill, int32_t* draft_tokens,
                     int32_t* draft_mask, int32_t* tokens, int32_t* mask, int32_t* k_star, int32_t* n_spec,
                     int32_t* n_comm, int32_t* sel, int32_t* n_sel, int32_t* sel_pos, cudaStream_t st,
                     const int32_t* pos, int32_t* status_dev) {
    StepTailArgs a;
    a.pos = pos;
    a.status_dev = status_dev;
    a.part_cap = part.cap;
    a.pm = part.m; a.ps = part.s; a.pa = part.a;
    a.plan = plan; a.n_rows = n_rows; a.M = M; a.p = p;
    a.tokV = tokV; a.confV = confV;
    a.sigma = sigma; a.n_fill = n_fill; a.draft_tokens = draft_tokens; a.draft_mask = draft_mask;
    a.tokens = tokens; a.mask = mask; a.k_star = k_star; a.n_spec = n_spec; a.n_comm = n_comm;
    a.sel = sel; a.n_sel = n_sel; a.sel_pos = sel_pos;
    // a multiple of 256 threads (merge groups), at least one thread per slot and per chain node
    int need = M > p.depth ? M : p.depth;
    int t = ((need + kCombineThreads - 1) / kCombineThreads) * kCombineThreads;
    const int rows_per_block = p.depth * M;
    while (t < 1024 && t * 2 <= 1024 && rows_per_block > (t / kCombineThreads) * kCombineRows) t *= 2;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(B);
    cfg.blockDim = dim3(t);
    cfg.dynamicSmemBytes = (size_t)t * 12;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = pdl_enabled() ? 1 : 0;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, step_tail_kernel, a);
    count_launch();
    return e == cudaSuccess ? PSD_OK : PSD_ERR_CUDA;
}

}  // namespace psd
