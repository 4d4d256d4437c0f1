// Draft construction and hierarchical acceptance for a general draft graph (Sec. 3.2 Stages 2-3;
// Algorithm 1 with a multi-parent DAG).  A node is a set of RANKS of the speculative ordering sigma
// (bit j of its 64-bit word = "speculate sigma_{j+1}"); an edge (p, k) needs S_p to be a strict subset
// of S_k, and by default every such pair is an edge, as the paper defines the edge set.
//
// Acceptance uses the fact that a speculated slot carries the same token in every draft that fills it
// (the cached step-t prediction, Eq. (2)), so whether slot sigma_j passes A_pi against parent p does
// not depend on the child: one 64-bit "pass" word per parent, built with warp votes, turns the
// per-edge check into   (S_k \ S_p) & ~pass[p] == 0.   One warp then walks the nodes in topological
// order, its lanes trying the accepted parents of a node in parallel.
#include "policy_common.cuh"

namespace psd {
namespace {

struct DagDev {
    int K;
    uint64_t ranks[PSD_MAX_DAG_NODES];
    uint64_t parents[PSD_MAX_DAG_NODES];
    int8_t topo[PSD_MAX_DAG_NODES];          // nodes by (number of ranks, index)
    int8_t node_with_rank[PSD_MAX_DAG_NODES]; // some node that speculates rank j, or -1
};

__device__ __forceinline__ uint64_t valid_ranks(int m) { return m >= 64 ? ~0ull : ((1ull << m) - 1ull); }

__global__ void build_dag_kernel(const float* __restrict__ conf, const int32_t* __restrict__ tok,
                                 const int32_t* __restrict__ node, int n_nodes_in,
                                 const int32_t* __restrict__ tokens, const int32_t* __restrict__ mask, int M,
                                 const DagDev g, int32_t* __restrict__ sigma, int32_t* __restrict__ n_fill,
                                 int32_t* __restrict__ draft_tokens, int32_t* __restrict__ draft_mask) {
    extern __shared__ unsigned char smem_raw[];
    float* s_conf = reinterpret_cast<float*>(smem_raw);
    int* s_flag = reinterpret_cast<int*>(s_conf + blockDim.x);
    const int b = blockIdx.x, i = threadIdx.x, K = g.K;
    const bool in = i < M;
    int nd = node ? node[b] : 0;
    nd = min(max(nd, 0), n_nodes_in - 1);
    const size_t src = ((size_t)b * n_nodes_in + nd) * M;
    const size_t st = (size_t)b * M;
    const float c = in ? conf[src + i] : 0.f;
    const int mk = in ? (mask[st + i] != 0) : 0;
    s_conf[i] = c;
    s_flag[i] = mk;
    const int m = __syncthreads_count(mk);
    int rank = M;
    if (mk) {
        rank = rank_among(s_conf, s_flag, M, c, i);
    }
    if (in && i >= m) sigma[st + i] = -1;
    if (mk) sigma[st + rank] = i;
    const uint64_t valid = valid_ranks(m);
    const int32_t cur = in ? tokens[st + i] : 0;
    const int32_t pred = mk ? tok[src + i] : 0;
    for (int k = 0; k < K; ++k) {
        if (i == 0) n_fill[(size_t)b * K + k] = __popcll(g.ranks[k] & valid);
        if (in) {
            const bool fill = mk && rank < 64 && ((g.ranks[k] >> rank) & 1ull);      // i in S_k
            const size_t o = ((size_t)b * K + k) * M + i;
            draft_tokens[o] = fill ? pred : cur;       // Eq. (2)
            draft_mask[o] = (mk && !fill) ? 1 : 0;
        }
    }
}

__global__ void accept_dag_kernel(const int32_t* __restrict__ tokV, const float* __restrict__ confV,
                                  const int32_t* __restrict__ sigma, const int32_t* __restrict__ draft_tokens,
                                  const int32_t* __restrict__ draft_mask, int M, psd_policy_t p, const DagDev g,
                                  int32_t* __restrict__ tokens, int32_t* __restrict__ mask,
                                  int32_t* __restrict__ k_star, int32_t* __restrict__ n_spec,
                                  int32_t* __restrict__ n_comm, int32_t* __restrict__ accepted) {
    __shared__ uint32_t s_pass[PSD_MAX_DAG_NODES][2];
    __shared__ unsigned long long s_acc;
    __shared__ int s_best;
    const int b = blockIdx.x, K = g.K;
    const size_t st = (size_t)b * M;
    const size_t blk = (size_t)b * K * M;

    int have = 0;
    for (int i = threadIdx.x; i < M; i += blockDim.x) have += sigma[st + i] >= 0;
    __shared__ int s_m;
    if (threadIdx.x == 0) s_m = 0;
    __syncthreads();
    if (have) atomicAdd(&s_m, have);
    __syncthreads();
    const int m_res = s_m;                       // residual masked slots = valid ranks
    const int n_ranks = min(m_res, 64);

    // pass[p] bit j: slot sigma_j passes A_pi against node p's predictions
    for (int item = threadIdx.x; item < K * 64; item += blockDim.x) {
        const int q = item >> 6, j = item & 63;
        bool ok = false;
        const int holder = j < n_ranks ? g.node_with_rank[j] : -1;
        if (holder >= 0) {
            const int i = sigma[st + j];
            const size_t po = blk + (size_t)q * M;
            const bool agree = tokV[po + i] == draft_tokens[blk + (size_t)holder * M + i];
            if (p.accept_mode == PSD_ACCEPT_AGREE_ONLY) {
                ok = agree;
            } else if (p.accept_mode == PSD_ACCEPT_AGREE_AND_CONF) {
                ok = agree && confV[po + i] > p.tau;
            } else {
                // the policy on node q's draft: is slot i among the positions it would commit?
                const float ci = confV[po + i];
                const bool mi = draft_mask[po + i] != 0;
                int n_masked = 0, n_thr = 0, rk = 0;
                for (int t = 0; t < M; ++t) {
                    const bool mt = draft_mask[po + t] != 0;
                    const float ct = confV[po + t];
                    n_masked += mt;
                    n_thr += mt && ct > p.tau;
                    rk += mt && ranks_before(ct, t, ci, i);
                }
                ok = agree && mi && rk < policy_count(n_thr, n_masked, p);
            }
        }
        const uint32_t bits = __ballot_sync(0xffffffffu, ok);
        if ((threadIdx.x & 31) == 0) s_pass[q][(j >> 5) & 1] = bits;
    }
    __syncthreads();

    // one warp walks the nodes in topological order; lanes try the parents
    if (threadIdx.x < 32) {
        const int lane = threadIdx.x;
        const uint64_t valid = valid_ranks(m_res);
        unsigned long long acc = 1ull;            // the root
        for (int t = 0; t < K; ++t) {
            const int k = g.topo[t];
            if (k == 0) continue;
            const uint64_t need = g.ranks[k] & valid;
            const uint64_t cand = g.parents[k] & acc;
            bool ok = false;
            for (int q = lane; q < K; q += 32) {
                if ((cand >> q) & 1ull) {
                    const uint64_t pass = ((uint64_t)s_pass[q][1] << 32) | (uint64_t)s_pass[q][0];
                    ok = ok || ((need & ~(g.ranks[q] & valid)) & ~pass) == 0ull;
                }
            }
            if (__any_sync(0xffffffffu, ok)) acc |= 1ull << k;
        }
        if (lane == 0) {
            int best = 0, best_n = -1;
            for (int k = 0; k < K; ++k) {
                const int n = __popcll(g.ranks[k] & valid);
                if (((acc >> k) & 1ull) && n > best_n) { best = k; best_n = n; }
            }
            s_acc = acc;
            s_best = best;
            k_star[b] = best;
            n_spec[b] = best_n;
        }
    }
    __syncthreads();
    const int best = s_best;
    int extra = 0;
    for (int i = threadIdx.x; i < M; i += blockDim.x) {
        const size_t o = blk + (size_t)best * M + i;
        int32_t t = draft_tokens[o];
        int mk = draft_mask[o] != 0;
        if (mk && confV[o] > p.tau) { t = tokV[o]; mk = 0; ++extra; }
        tokens[st + i] = t;
        mask[st + i] = mk;
    }
    __shared__ int s_extra;
    if (threadIdx.x == 0) s_extra = 0;
    __syncthreads();
    if (extra) atomicAdd(&s_extra, extra);
    __syncthreads();
    if (threadIdx.x == 0) n_comm[b] = n_spec[b] + s_extra;
    if (accepted)
        for (int k = threadIdx.x; k < K; k += blockDim.x) accepted[(size_t)b * K + k] = (int)((s_acc >> k) & 1ull);
}

// Checks a graph and prepares its device form.  Returns PSD_OK or PSD_ERR_SHAPE.
int prepare(const psd_dag_t* g, DagDev* d) {
    if (g->n_nodes < 1 || g->n_nodes > PSD_MAX_DAG_NODES || g->ranks[0] != 0) return PSD_ERR_SHAPE;
    const int K = g->n_nodes;
    d->K = K;
    for (int j = 0; j < 64; ++j) d->node_with_rank[j] = -1;
    for (int k = 0; k < K; ++k) {
        d->ranks[k] = g->ranks[k];
        d->parents[k] = g->parents[k];
        if (K < 64 && (g->parents[k] >> K) != 0) return PSD_ERR_SHAPE;
        for (int q = 0; q < K; ++q)
            if ((g->parents[k] >> q) & 1ull) {
                // an edge (q, k) needs S_q to be a strict subset of S_k
                if ((g->ranks[q] & ~g->ranks[k]) != 0 || g->ranks[q] == g->ranks[k]) return PSD_ERR_SHAPE;
            }
        for (int j = 0; j < 64; ++j)
            if (((g->ranks[k] >> j) & 1ull) && d->node_with_rank[j] < 0) d->node_with_rank[j] = (int8_t)k;
    }
    for (int k = K; k < PSD_MAX_DAG_NODES; ++k) { d->ranks[k] = 0; d->parents[k] = 0; }
    // topological order: fewer ranks first, lower index first among equals (a strict subset has fewer ranks)
    int n = 0;
    for (int c = 0; c <= 64; ++c)
        for (int k = 0; k < K; ++k)
            if (__builtin_popcountll(g->ranks[k]) == c) d->topo[n++] = (int8_t)k;
    for (int k = n; k < PSD_MAX_DAG_NODES; ++k) d->topo[k] = 0;
    return PSD_OK;
}

inline int block_threads(int M) { return ((M + 31) / 32) * 32; }

}  // namespace
}  // namespace psd

using namespace psd;

extern "C" {

int psd_dag_init(psd_dag_t* g, int32_t n_nodes, const uint64_t* ranks, const uint64_t* parents) {
    if (!g || !ranks) return PSD_ERR_NULL;
    if (n_nodes < 1 || n_nodes > PSD_MAX_DAG_NODES || ranks[0] != 0) return PSD_ERR_SHAPE;
    g->n_nodes = n_nodes;
    g->reserved = 0;
    for (int k = 0; k < PSD_MAX_DAG_NODES; ++k) {
        g->ranks[k] = k < n_nodes ? ranks[k] : 0;
        g->parents[k] = 0;
    }
    for (int k = 0; k < n_nodes; ++k) {
        if (parents) {
            g->parents[k] = parents[k];
        } else {
            for (int q = 0; q < n_nodes; ++q)
                if ((ranks[q] & ~ranks[k]) == 0 && ranks[q] != ranks[k]) g->parents[k] |= 1ull << q;
        }
    }
    DagDev d;
    return prepare(g, &d);
}

int psd_build_drafts_dag(const float* conf, const int32_t* tok, const int32_t* node, int32_t n_nodes,
                         const int32_t* tokens, const int32_t* mask, int32_t B, int32_t M, psd_policy_t p,
                         const psd_dag_t* g, int32_t* sigma, int32_t* n_fill, int32_t* draft_tokens,
                         int32_t* draft_mask, void* cuda_stream) {
    (void)p;
    if (!conf || !tok || !tokens || !mask || !g || !sigma || !n_fill || !draft_tokens || !draft_mask) return PSD_ERR_NULL;
    if (B < 1 || M < 1 || M > PSD_MAX_M || n_nodes < 1 || n_nodes > PSD_MAX_DEPTH) return PSD_ERR_SHAPE;
    DagDev d;
    if (int e = prepare(g, &d)) return e;
    const int t = block_threads(M);
    build_dag_kernel<<<B, t, (size_t)t * 8, reinterpret_cast<cudaStream_t>(cuda_stream)>>>(
        conf, tok, node, n_nodes, tokens, mask, M, d, sigma, n_fill, draft_tokens, draft_mask);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? PSD_OK : PSD_ERR_CUDA;
}

int psd_verify_accept_dag(const int32_t* tokV, const float* confV, const int32_t* sigma,
                          const int32_t* draft_tokens, const int32_t* draft_mask, int32_t B, int32_t M,
                          psd_policy_t p, const psd_dag_t* g, int32_t* tokens, int32_t* mask, int32_t* k_star,
                          int32_t* n_spec_accepted, int32_t* n_committed, int32_t* accepted, void* cuda_stream) {
    if (!tokV || !confV || !sigma || !draft_tokens || !draft_mask || !g || !tokens || !mask || !k_star ||
        !n_spec_accepted || !n_committed)
        return PSD_ERR_NULL;
    if (B < 1 || M < 1 || M > PSD_MAX_M) return PSD_ERR_SHAPE;
    if (p.k_min < 1 || (p.k_max != 0 && p.k_max < p.k_min) || p.accept_mode < 0 || p.accept_mode > 2 || p.tau != p.tau)
        return PSD_ERR_POLICY;
    DagDev d;
    if (int e = prepare(g, &d)) return e;
    int t = block_threads(M);
    if (t < 128) t = 128;
    accept_dag_kernel<<<B, t, 0, reinterpret_cast<cudaStream_t>(cuda_stream)>>>(
        tokV, confV, sigma, draft_tokens, draft_mask, M, p, d, tokens, mask, k_star, n_spec_accepted, n_committed,
        accepted);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? PSD_OK : PSD_ERR_CUDA;
}

}  // extern "C"
