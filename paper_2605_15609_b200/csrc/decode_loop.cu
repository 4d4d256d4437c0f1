// psd_decode_blocks: Algorithm 1 as a whole, for a batch of blocks, driven from the host.
//
// The transformer body is the caller's (a callback that turns token states into final hidden
// states on the device); everything after it runs in this library's kernels: psd_confidence,
// psd_select_unmask, psd_build_drafts, psd_verify_accept (or psd_step in the one-call-per-iteration
// order).  After every state update a small kernel counts the masked slots of every block; the host
// reads the total (one 4-byte copy and a stream synchronisation per check) and stops when no
// block has a masked slot left (Algorithm 1's while condition and its early break).
//
// psd_table_body is a stand-in body for tests and benchmarks: a table look-up with no arithmetic.
#include <cuda_bf16.h>
#include "psd_internal.cuh"

namespace psd {
namespace {

// One thread block per sequence block.  n_masked[b] still holds the count from the previous check:
// a block that had masked slots then has just been through `passes_since` forward passes.
// The blocks add their counts into counters[0]; the last block to finish (a ticket from counters[1])
// takes the sum, leaves both counters at zero for the next check, and publishes (sum, seq) as one
// 8-byte word: to `publish` when the host gave a mapped pinned word, and to counters[2..3] always.
__global__ void progress_kernel(const int32_t* __restrict__ mask, int M, int passes_since, int iteration,
                                int32_t* __restrict__ n_masked, int32_t* __restrict__ counters,
                                int32_t* __restrict__ passes, int32_t* __restrict__ done_iteration,
                                unsigned long long* publish, uint32_t seq) {
    const int b = blockIdx.x;
    int mine = 0;
    for (int i = threadIdx.x; i < M; i += blockDim.x) mine += mask[(size_t)b * M + i] != 0;
    __shared__ int s_sum;
    if (threadIdx.x == 0) s_sum = 0;
    __syncthreads();
    if (mine) atomicAdd(&s_sum, mine);
    __syncthreads();
    if (threadIdx.x == 0) {
        const int before = n_masked[b];
        if (before > 0 && passes) passes[b] += passes_since;
        if (before > 0 && s_sum == 0 && done_iteration) done_iteration[b] = iteration;
        n_masked[b] = s_sum;
        if (s_sum) atomicAdd(&counters[0], s_sum);
        __threadfence();
        if (atomicAdd(&counters[1], 1) == (int)gridDim.x - 1) {
            const int total = atomicExch(&counters[0], 0);
            counters[1] = 0;
            const unsigned long long word = ((unsigned long long)seq << 32) | (uint32_t)total;
            *reinterpret_cast<volatile unsigned long long*>(counters + 2) = word;
            if (publish) {
                *reinterpret_cast<volatile unsigned long long*>(publish) = word;
                __threadfence_system();
            }
        }
    }
}

// Drafts that are D copies of the state with nothing speculated (sigma empty, n_fill = 0): what the
// one-call-per-iteration order verifies in its first iteration.
__global__ void root_drafts_kernel(const int32_t* __restrict__ tokens, const int32_t* __restrict__ mask, int M, int D,
                                   int32_t* __restrict__ sigma, int32_t* __restrict__ n_fill,
                                   int32_t* __restrict__ draft_tokens, int32_t* __restrict__ draft_mask) {
    const int b = blockIdx.x;
    for (int i = threadIdx.x; i < M; i += blockDim.x) {
        const int32_t t = tokens[(size_t)b * M + i], m = mask[(size_t)b * M + i];
        sigma[(size_t)b * M + i] = -1;
        for (int d = 0; d < D; ++d) {
            draft_tokens[((size_t)b * D + d) * M + i] = t;
            draft_mask[((size_t)b * D + d) * M + i] = m;
        }
    }
    for (int d = threadIdx.x; d < D; d += blockDim.x) n_fill[(size_t)b * D + d] = 0;
}

__global__ void trace_kernel(const int32_t* __restrict__ n_sel, const int32_t* __restrict__ k_star,
                             const int32_t* __restrict__ n_spec, const int32_t* __restrict__ n_comm, int B,
                             int have_accept, int32_t* __restrict__ out) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    out[b * 4 + 0] = n_sel[b];
    out[b * 4 + 1] = have_accept ? k_star[b] : 0;
    out[b * 4 + 2] = have_accept ? n_spec[b] : 0;
    out[b * 4 + 3] = have_accept ? n_comm[b] : 0;
}

// hidden[(s, i), :] = table[((b * M + i) * 3 + c), :] with b = s / seq_per_block and c = the number of
// committed neighbours (slots i-1 and i+1 of the same sequence whose mask is 0).
__global__ void table_body_kernel(const uint4* __restrict__ table, const int32_t* __restrict__ mask, int M, int H,
                                  int seq_per_block, uint4* __restrict__ hidden) {
    const int row = blockIdx.x;            // (s, i)
    const int s = row / M, i = row - s * M;
    const int b = s / seq_per_block;
    const int32_t* mk = mask + (size_t)s * M;
    const int c = (i > 0 && mk[i - 1] == 0 ? 1 : 0) + (i + 1 < M && mk[i + 1] == 0 ? 1 : 0);
    const size_t src = ((size_t)(b * M + i) * 3 + c) * (size_t)(H / 8);
    const size_t dst = (size_t)row * (size_t)(H / 8);
    for (int j = threadIdx.x; j < H / 8; j += blockDim.x) hidden[dst + j] = table[src + j];
}

// A pinned, mapped 8-byte word per host thread through which the progress kernel hands the host its
// result without a copy operation (allocated on the thread's first call, kept until the process exits).
// NULL if the allocation fails: the result is then copied from the device counters instead.
unsigned long long* host_word() {
    thread_local unsigned long long* word = nullptr;
    thread_local bool tried = false;
    if (!tried) {
        tried = true;
        void* p = nullptr;
        if (cudaHostAlloc(&p, 64, cudaHostAllocPortable | cudaHostAllocMapped) == cudaSuccess) {
            word = reinterpret_cast<unsigned long long*>(p);
            *word = 0;
        } else {
            (void)cudaGetLastError();
        }
    }
    return word;
}

// Waits for the stream and returns the sum the progress kernel published with sequence number `seq`.
int read_total(int32_t* counters, unsigned long long* word, uint32_t seq, cudaStream_t st, int* out) {
    unsigned long long v = 0;
    if (word) {
        if (cudaStreamSynchronize(st) != cudaSuccess) return PSD_ERR_CUDA;
        v = *reinterpret_cast<volatile unsigned long long*>(word);
    }
    if (!word || (uint32_t)(v >> 32) != seq) {
        // no mapped word (or the write has not arrived, which a finished stream rules out): copy the device's
        if (cudaMemcpyAsync(&v, counters + 2, 8, cudaMemcpyDeviceToHost, st) != cudaSuccess) return PSD_ERR_CUDA;
        if (cudaStreamSynchronize(st) != cudaSuccess) return PSD_ERR_CUDA;
        if ((uint32_t)(v >> 32) != seq) return PSD_ERR_CUDA;
    }
    *out = (int)(uint32_t)v;
    return PSD_OK;
}

}  // namespace
}  // namespace psd

using namespace psd;

extern "C" {

int psd_table_body(void* user, const int32_t* tokens, const int32_t* mask, int32_t n_seq, int32_t M,
                   void* hidden_bf16, void* cuda_stream) {
    (void)tokens;
    const psd_table_body_t* t = reinterpret_cast<const psd_table_body_t*>(user);
    if (!t || !t->table_bf16 || !mask || !hidden_bf16) return PSD_ERR_NULL;
    if (t->B < 1 || n_seq < t->B || n_seq % t->B != 0 || M < 1 || t->H < 8 || t->H % 8 != 0) return PSD_ERR_SHAPE;
    if ((reinterpret_cast<uintptr_t>(t->table_bf16) & 15) || (reinterpret_cast<uintptr_t>(hidden_bf16) & 15))
        return PSD_ERR_ALIGN;
    table_body_kernel<<<n_seq * M, 128, 0, reinterpret_cast<cudaStream_t>(cuda_stream)>>>(
        reinterpret_cast<const uint4*>(t->table_bf16), mask, M, t->H, n_seq / t->B,
        reinterpret_cast<uint4*>(hidden_bf16));
    count_launch();
    return cudaGetLastError() == cudaSuccess ? PSD_OK : PSD_ERR_CUDA;
}

size_t psd_decode_scratch_bytes(int32_t B, int32_t M) {
    if (B < 1 || M < 1 || M > PSD_MAX_M) return 0;
    // n_masked[B] (rounded up to a multiple of 8 bytes), counters[4], tok1[B*M], conf1[B*M]
    return (((size_t)B * 4 + 7) / 8 * 8 + 16 + (size_t)B * M * 8 + 255) / 256 * 256;
}

int psd_decode_blocks(psd_body_fn body, void* user, const psd_step_io_t* io, int32_t B, int32_t M, int32_t H,
                      int32_t V, psd_policy_t p, const psd_dag_t* g, int32_t order, int32_t max_iterations,
                      void* scratch, size_t scratch_bytes, void* workspace, size_t workspace_bytes,
                      int32_t* status_dev, int32_t* passes, int32_t* done_iteration, int32_t* trace,
                      psd_decode_stats_t* stats, void* cuda_stream) {
    if (!body || !io || !scratch || !workspace || !stats) return PSD_ERR_NULL;
    if (!io->hidden_bf16 || !io->w_lm_bf16 || !io->sigma || !io->n_fill || !io->draft_tokens || !io->draft_mask ||
        !io->tokV || !io->confV || !io->tokens || !io->mask || !io->k_star || !io->n_spec_accepted ||
        !io->n_committed || !io->sel || !io->n_sel || !io->sel_pos)
        return PSD_ERR_NULL;
    if (order != PSD_ORDER_TWO_PASSES && order != PSD_ORDER_ONE_PASS) return PSD_ERR_UNSUPPORTED;
    if (max_iterations < 1) return PSD_ERR_SHAPE;
    const size_t need = psd_decode_scratch_bytes(B, M);
    if (need == 0) return PSD_ERR_SHAPE;
    if (reinterpret_cast<uintptr_t>(scratch) & 255) return PSD_ERR_ALIGN;
    if (scratch_bytes < need) return PSD_ERR_WORKSPACE;
    if (g) {
        if (g->n_nodes < 1 || g->n_nodes > PSD_MAX_DAG_NODES) return PSD_ERR_SHAPE;
        p.depth = g->n_nodes;     // the drafts are the nodes of the graph
    }
    const int D = p.depth;
    if (D < 1 || D > PSD_MAX_DEPTH || (long long)B * D * M > 2147483647ll) return PSD_ERR_POLICY;
    if (workspace_bytes < psd_workspace_bytes(B * D * M, H, V) || psd_workspace_bytes(B * D * M, H, V) == 0)
        return PSD_ERR_WORKSPACE;

    cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
    int32_t* n_masked = reinterpret_cast<int32_t*>(scratch);
    int32_t* counters = n_masked + (B + 1) / 2 * 2;   // 8-byte aligned: [sum, tickets, published word (2)]
    int32_t* tok1 = counters + 4;
    float* conf1 = reinterpret_cast<float*>(tok1 + (size_t)B * M);
    void* hidden = const_cast<void*>(io->hidden_bf16);
    const int threads = M < 256 ? ((M + 31) / 32) * 32 : 256;

    stats->iterations = 0;
    stats->forward_passes = 0;
    stats->masked_left = 0;
    bool ok = true;
    auto cuda_ok = [&](cudaError_t e) { ok = ok && e == cudaSuccess; };
    unsigned long long* word = host_word();
    unsigned long long* word_dev = nullptr;
    if (word && cudaHostGetDevicePointer(reinterpret_cast<void**>(&word_dev), word, 0) != cudaSuccess) {
        (void)cudaGetLastError();
        word = nullptr;
        word_dev = nullptr;
    }
    uint32_t seq = word ? (uint32_t)(*word >> 32) : 0u;   // continues this thread's numbering
    auto progress = [&](int passes_since, int iteration, int* masked_now) -> int {
        ++seq;
        progress_kernel<<<B, threads, 0, st>>>(io->mask, M, passes_since, iteration, n_masked, counters, passes,
                                               done_iteration, word_dev, seq);
        count_launch();
        cuda_ok(cudaGetLastError());
        if (!ok) return PSD_ERR_CUDA;
        return read_total(counters, word, seq, st, masked_now);
    };
    auto record = [&](int iteration, int have_accept) {
        if (!trace) return;
        trace_kernel<<<(B + 127) / 128, 128, 0, st>>>(io->n_sel, io->k_star, io->n_spec_accepted, io->n_committed, B,
                                                      have_accept, trace + (size_t)iteration * B * 4);
        count_launch();
    };

    // the blocks' state as the caller left it: count it once, charge no pass
    cuda_ok(cudaMemsetAsync(n_masked, 0, (size_t)((B + 1) / 2 * 2 + 4) * 4, st));   // counts and counters
    if (passes) cuda_ok(cudaMemsetAsync(passes, 0, (size_t)B * 4, st));
    if (done_iteration) cuda_ok(cudaMemsetAsync(done_iteration, 0xFF, (size_t)B * 4, st));
    int masked = 0;
    if (int e = progress(0, 0, &masked)) return e;

    int e = PSD_OK;
    if (order == PSD_ORDER_ONE_PASS && masked > 0) {
        root_drafts_kernel<<<B, threads, 0, st>>>(io->tokens, io->mask, M, D, io->sigma, io->n_fill, io->draft_tokens,
                                                  io->draft_mask);
        count_launch();
    }
    int it = 0;
    while (masked > 0 && it < max_iterations) {
        if (order == PSD_ORDER_ONE_PASS) {
            // one forward pass per iteration: the verification pass of the drafts doubles as the model
            // call of the next iteration (psd_step)
            if ((e = body(user, io->draft_tokens, io->draft_mask, B * D, M, hidden, cuda_stream))) return e;
            e = g ? psd_step_dag(io, B, M, H, V, p, g, workspace, workspace_bytes, status_dev, cuda_stream)
                  : psd_step(io, B, M, H, V, p, workspace, workspace_bytes, status_dev, cuda_stream);
            if (e) return e;
            stats->forward_passes += 1;
            record(it, 1);
            if ((e = progress(1, it, &masked))) return e;
        } else {
            // Algorithm 1 as printed.  Stage 1: one pass on the current state, policy, Eq. (1).
            if ((e = body(user, io->tokens, io->mask, B, M, hidden, cuda_stream))) return e;
            e = psd_compact_rows_enabled(B * M)
                    ? psd_confidence_masked(hidden, io->w_lm_bf16, io->mask, B * M, H, V, tok1, conf1, nullptr,
                                            workspace, workspace_bytes, status_dev, cuda_stream)
                    : psd_confidence(hidden, io->w_lm_bf16, nullptr, B * M, H, V, tok1, conf1, nullptr, workspace,
                                     workspace_bytes, status_dev, cuda_stream);
            if (e) return e;
            if ((e = psd_select_unmask(conf1, tok1, nullptr, 1, io->tokens, io->mask, B, M, p, io->sel, io->n_sel,
                                       io->sel_pos, cuda_stream)))
                return e;
            stats->forward_passes += 1;
            if ((e = progress(1, it, &masked))) return e;
            if (masked == 0 || D == 1) {
                // every block is resolved (the early break), or the chain is the root alone and there is
                // nothing to speculate: plain spatial decoding
                record(it, 0);
            } else {
                // Stage 2: drafts from the cached stage-1 predictions.  Stage 3: one batched pass, acceptance.
                e = g ? psd_build_drafts_dag(conf1, tok1, nullptr, 1, io->tokens, io->mask, B, M, p, g, io->sigma,
                                             io->n_fill, io->draft_tokens, io->draft_mask, cuda_stream)
                      : psd_build_drafts(conf1, tok1, nullptr, 1, io->tokens, io->mask, B, M, p, io->sigma,
                                         io->n_fill, io->draft_tokens, io->draft_mask, cuda_stream);
                if (e) return e;
                if ((e = body(user, io->draft_tokens, io->draft_mask, B * D, M, hidden, cuda_stream))) return e;
                e = psd_compact_rows_enabled(B * D * M)
                        ? psd_confidence_masked(hidden, io->w_lm_bf16, io->draft_mask, B * D * M, H, V, io->tokV,
                                                io->confV, nullptr, workspace, workspace_bytes, status_dev,
                                                cuda_stream)
                        : psd_confidence(hidden, io->w_lm_bf16, nullptr, B * D * M, H, V, io->tokV, io->confV,
                                         nullptr, workspace, workspace_bytes, status_dev, cuda_stream);
                if (e) return e;
                e = g ? psd_verify_accept_dag(io->tokV, io->confV, io->sigma, io->draft_tokens, io->draft_mask, B, M,
                                              p, g, io->tokens, io->mask, io->k_star, io->n_spec_accepted,
                                              io->n_committed, nullptr, cuda_stream)
                      : psd_verify_accept(io->tokV, io->confV, io->sigma, io->n_fill, io->draft_tokens,
                                          io->draft_mask, B, M, p, io->tokens, io->mask, io->k_star,
                                          io->n_spec_accepted, io->n_committed, nullptr, cuda_stream);
                if (e) return e;
                stats->forward_passes += 1;
                record(it, 1);
                if ((e = progress(1, it, &masked))) return e;
            }
        }
        ++it;
    }
    if (!ok) return PSD_ERR_CUDA;
    stats->iterations = it;
    stats->masked_left = masked;
    return PSD_OK;
}

}  // extern "C"
