// extern "C" entry points of libpsd_b200: argument checking, then kernel launches.  See psd.h.
#include <atomic>
#include <cmath>
#include <cstring>
#include <mutex>
#include "psd_internal.cuh"

namespace psd {
namespace {
std::atomic<long long> g_launches{0};
std::atomic<int> g_conf_impl{0};
std::atomic<int> g_pdl{1};
std::atomic<int> g_band_bytes{36 << 20};
std::atomic<int> g_tile_order{0};
std::atomic<int> g_compact{0};
std::atomic<int> g_wait_kcycles{4000000};   // thousands of clock cycles: about 2 s
std::atomic<int> g_stall_test{0};
thread_local cudaEvent_t t_ev_start = nullptr, t_ev_stop = nullptr;

inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }
inline size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

int check_policy(const psd_policy_t& p) {
    if (p.k_min < 1 || (p.k_max != 0 && p.k_max < p.k_min) || p.depth < 1 || p.depth > PSD_MAX_DEPTH ||
        p.stride < 0 || p.accept_mode < 0 || p.accept_mode > 2 || std::isnan(p.tau))
        return PSD_ERR_POLICY;
    return PSD_OK;
}

int check_block_shape(int B, int M) { return (B < 1 || M < 1 || M > PSD_MAX_M) ? PSD_ERR_SHAPE : PSD_OK; }

bool conf_shape_ok(int n_rows, int H, int V) {
    return n_rows >= 1 && H >= 64 && H % 64 == 0 && V >= 1 && V < 2147483647 - 256;
}
}  // namespace

// Default choice by measurement (V = 126464, H = 4096): see launch_confidence_tc.
static bool confidence_uses_pairs(int impl, int n_rows) {
    return impl == 3 || (impl == 0 && n_rows > 128 && n_rows <= 256);
}

void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }
int pdl_enabled() { return g_pdl.load(std::memory_order_relaxed); }
long long band_bytes() { return g_band_bytes.load(std::memory_order_relaxed); }
int tile_order() { return g_tile_order.load(std::memory_order_relaxed); }
long long wait_limit_cycles() { return 1000ll * g_wait_kcycles.load(std::memory_order_relaxed); }
int selftest_stall() { return g_stall_test.load(std::memory_order_relaxed); }

int launch_confidence(const void* hidden, const void* w, int n_rows, int H, int V, Partials part,
                      int32_t* status_dev, cudaStream_t st, SplitPlan* plan, const int32_t* n_rows_dev) {
    const int impl = g_conf_impl.load(std::memory_order_relaxed);
    if (impl == 1) {
        // the CUDA-core cross-check kernel scores every row of the buffer, whatever the device-side count
        const int n_split = launch_confidence_simt(hidden, w, n_rows, H, V, part, st);
        if (n_split < 0) return n_split;
        *plan = uniform_splits(n_split);
        return PSD_OK;
    }
    // Default choice by measurement (V = 126464, H = 4096): at 129..256 rows one CTA pair covers both row
    // tiles and fetches every W tile once (258-265 us against 276-282 us); at 128 rows and below, and
    // from 257 rows up, the single-CTA kernel is faster or equal (see confidence_tc2.cu).
    const bool pairs = confidence_uses_pairs(impl, n_rows);
    return pairs ? launch_confidence_tc2(hidden, w, n_rows, H, V, part, status_dev, n_rows_dev, st, plan)
                 : launch_confidence_tc1(hidden, w, n_rows, H, V, part, status_dev, n_rows_dev, st, plan);
}
}  // namespace psd

using namespace psd;

extern "C" {

const char* psd_status_string(int code) {
    switch (code) {
        case PSD_OK: return "ok";
        case PSD_ERR_NULL: return "a required pointer is NULL";
        case PSD_ERR_SHAPE: return "a size is out of range";
        case PSD_ERR_ALIGN: return "a pointer is not sufficiently aligned";
        case PSD_ERR_WORKSPACE: return "workspace too small";
        case PSD_ERR_POLICY: return "invalid policy parameters";
        case PSD_ERR_CUDA: return "a CUDA call failed";
        case PSD_ERR_UNSUPPORTED: return "a reserved argument was used";
        case PSD_ERR_TIMEOUT: return "a bounded wait inside a kernel expired";
        case PSD_ERR_INTERNAL: return "a debug-build check inside a kernel failed";
        default: return "unknown status";
    }
}

size_t psd_workspace_bytes(int32_t n_rows, int32_t H, int32_t V) {
    if (!conf_shape_ok(n_rows, H, V)) return 0;
    return round_up((size_t)max_splits(V) * (size_t)n_rows * 12, 256);
}

size_t psd_compact_workspace_bytes(int32_t n_rows, int32_t H, int32_t V) {
    if (!conf_shape_ok(n_rows, H, V)) return 0;
    return partial_bytes(n_rows, V) + compact_extra_bytes(n_rows, H);
}

int psd_compact_rows_enabled(int32_t n_rows) {
    const int mode = g_compact.load(std::memory_order_relaxed);
    return (mode == 2 || (mode == 1 && n_rows > 128)) ? 1 : 0;
}

int psd_set_confidence_impl(int impl) {
    if (impl < 0 || impl > 3) return PSD_ERR_SHAPE;
    return g_conf_impl.exchange(impl);
}

int psd_set_tuning(int knob, int value) {
    switch (knob) {
        case PSD_TUNE_BAND_BYTES:
            if (value < 0) return PSD_ERR_SHAPE;
            g_band_bytes.store(value);
            return PSD_OK;
        case PSD_TUNE_TILE_ORDER:
            if (value < 0 || value > 2) return PSD_ERR_SHAPE;
            g_tile_order.store(value);
            return PSD_OK;
        case PSD_TUNE_COMPACT_ROWS:
            if (value < 0 || value > 2) return PSD_ERR_SHAPE;
            g_compact.store(value);
            return PSD_OK;
        case PSD_TUNE_WAIT_LIMIT:
            if (value < 1) return PSD_ERR_SHAPE;
            g_wait_kcycles.store(value);
            return PSD_OK;
        case PSD_TUNE_SELFTEST_STALL:
            if (value != 0 && value != 1) return PSD_ERR_SHAPE;
            g_stall_test.store(value);
            return PSD_OK;
        case PSD_TUNE_PDL:
            if (value < 0 || value > 2) return PSD_ERR_SHAPE;
            g_pdl.store(value);
            return PSD_OK;
        default:
            return PSD_ERR_UNSUPPORTED;
    }
}

int psd_set_kernel_events(void* start_event, void* stop_event) {
    t_ev_start = reinterpret_cast<cudaEvent_t>(start_event);
    t_ev_stop = reinterpret_cast<cudaEvent_t>(stop_event);
    return PSD_OK;
}

const char* psd_confidence_kernel_name(int32_t n_rows) {
    const int impl = g_conf_impl.load(std::memory_order_relaxed);
    if (impl == 1) return "confidence_simt_kernel";
    return confidence_uses_pairs(impl, n_rows) ? "confidence_tc2_kernel" : "confidence_tc_kernel";
}

int64_t psd_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

int psd_confidence(const void* hidden_bf16, const void* w_lm_bf16, const int32_t* row_ids,
                   int32_t n_rows, int32_t H, int32_t V,
                   int32_t* out_token, float* out_conf, float* out_lse,
                   void* workspace, size_t workspace_bytes, int32_t* status_dev, void* cuda_stream) {
    if (!hidden_bf16 || !w_lm_bf16 || !out_token || !out_conf || !workspace) return PSD_ERR_NULL;
    if (!conf_shape_ok(n_rows, H, V)) return PSD_ERR_SHAPE;
    if (!aligned(hidden_bf16, 16) || !aligned(w_lm_bf16, 16) || !aligned(workspace, 256) ||
        !aligned(out_token, 4) || !aligned(out_conf, 4) || !aligned(out_lse, 4) || !aligned(status_dev, 4) ||
        !aligned(row_ids, 4))
        return PSD_ERR_ALIGN;
    if (workspace_bytes < (row_ids ? psd_compact_workspace_bytes(n_rows, H, V) : psd_workspace_bytes(n_rows, H, V)))
        return PSD_ERR_WORKSPACE;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
    Partials part = carve_partials(workspace, n_rows, V);
    if (row_ids) {
        // the listed rows are copied into a dense buffer first; everything after is the dense path
        CompactSpace cs = carve_compact(workspace, n_rows, H, V);
        if (int e = launch_gather_rows(hidden_bf16, row_ids, nullptr, n_rows, n_rows, H, cs.hidden, st)) return e;
        hidden_bf16 = cs.hidden;
    }
    const bool timed = t_ev_start && t_ev_stop;
    if (timed && cudaEventRecord(t_ev_start, st) != cudaSuccess) return PSD_ERR_CUDA;
    SplitPlan plan;
    const int rc = launch_confidence(hidden_bf16, w_lm_bf16, n_rows, H, V, part, status_dev, st, &plan);
    if (timed) {
        cudaError_t e = cudaEventRecord(t_ev_stop, st);
        t_ev_start = t_ev_stop = nullptr;
        if (e != cudaSuccess) return PSD_ERR_CUDA;
    }
    if (rc < 0) return rc;
    return launch_combine(part, plan, n_rows, out_token, out_conf, out_lse, st, nullptr, nullptr, 0, status_dev);
}

int psd_confidence_masked(const void* hidden_bf16, const void* w_lm_bf16, const int32_t* row_mask,
                          int32_t n_rows, int32_t H, int32_t V,
                          int32_t* out_token, float* out_conf, float* out_lse,
                          void* workspace, size_t workspace_bytes, int32_t* status_dev, void* cuda_stream) {
    if (!hidden_bf16 || !w_lm_bf16 || !row_mask || !out_token || !out_conf || !workspace) return PSD_ERR_NULL;
    if (!conf_shape_ok(n_rows, H, V)) return PSD_ERR_SHAPE;
    if (!aligned(hidden_bf16, 16) || !aligned(w_lm_bf16, 16) || !aligned(workspace, 256) || !aligned(row_mask, 4) ||
        !aligned(out_token, 4) || !aligned(out_conf, 4) || !aligned(out_lse, 4) || !aligned(status_dev, 4))
        return PSD_ERR_ALIGN;
    if (workspace_bytes < psd_compact_workspace_bytes(n_rows, H, V)) return PSD_ERR_WORKSPACE;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
    Partials part = carve_partials(workspace, n_rows, V);
    CompactSpace cs = carve_compact(workspace, n_rows, H, V);
    // list the flagged rows, copy them into a dense buffer, score as many rows as the device-side count
    // says, and merge every flagged row's partials back to the row's own place
    if (int e = launch_list_rows(row_mask, n_rows, cs.row_ids, cs.pos, cs.count, st)) return e;
    if (int e = launch_gather_rows(hidden_bf16, cs.row_ids, cs.count, 0, n_rows, H, cs.hidden, st)) return e;
    const bool timed = t_ev_start && t_ev_stop;
    if (timed && cudaEventRecord(t_ev_start, st) != cudaSuccess) return PSD_ERR_CUDA;
    SplitPlan plan;
    const int rc = launch_confidence(cs.hidden, w_lm_bf16, n_rows, H, V, part, status_dev, st, &plan, cs.count);
    if (timed) {
        cudaError_t e = cudaEventRecord(t_ev_stop, st);
        t_ev_start = t_ev_stop = nullptr;
        if (e != cudaSuccess) return PSD_ERR_CUDA;
    }
    if (rc < 0) return rc;
    return launch_combine(part, plan, n_rows, out_token, out_conf, out_lse, st, cs.pos, nullptr, 0, status_dev);
}

int psd_confidence_partial(const void* hidden_bf16, const void* w_shard_bf16, int32_t n_rows, int32_t H,
                           int32_t V_shard, int32_t v_offset, float* out_max, float* out_sumexp, int32_t* out_arg,
                           void* workspace, size_t workspace_bytes, int32_t* status_dev, void* cuda_stream) {
    if (!hidden_bf16 || !w_shard_bf16 || !out_max || !out_sumexp || !out_arg || !workspace) return PSD_ERR_NULL;
    if (!conf_shape_ok(n_rows, H, V_shard) || v_offset < 0 || (long long)v_offset + V_shard > 2147483647ll - 256)
        return PSD_ERR_SHAPE;
    if (!aligned(hidden_bf16, 16) || !aligned(w_shard_bf16, 16) || !aligned(workspace, 256) || !aligned(out_max, 4) ||
        !aligned(out_sumexp, 4) || !aligned(out_arg, 4) || !aligned(status_dev, 4))
        return PSD_ERR_ALIGN;
    if (workspace_bytes < psd_workspace_bytes(n_rows, H, V_shard)) return PSD_ERR_WORKSPACE;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
    Partials part = carve_partials(workspace, n_rows, V_shard);
    SplitPlan plan;
    if (int rc = launch_confidence(hidden_bf16, w_shard_bf16, n_rows, H, V_shard, part, status_dev, st, &plan)) return rc;
    return launch_combine(part, plan, n_rows, out_arg, out_sumexp, nullptr, st, nullptr, out_max, v_offset, status_dev);
}

int psd_merge_partials(const float* max, const float* sumexp, const int32_t* arg, int32_t n_shards, int32_t n_rows,
                       int32_t* out_token, float* out_conf, float* out_lse, void* cuda_stream) {
    if (!max || !sumexp || !arg || !out_token || !out_conf) return PSD_ERR_NULL;
    if (n_shards < 1 || n_rows < 1) return PSD_ERR_SHAPE;
    if (!aligned(max, 4) || !aligned(sumexp, 4) || !aligned(arg, 4) || !aligned(out_token, 4) ||
        !aligned(out_conf, 4) || !aligned(out_lse, 4))
        return PSD_ERR_ALIGN;
    Partials part;
    part.m = const_cast<float*>(max);
    part.s = const_cast<float*>(sumexp);
    part.a = const_cast<int32_t*>(arg);
    part.cap = (size_t)n_shards * (size_t)n_rows;
    return launch_combine(part, uniform_splits(n_shards), n_rows, out_token, out_conf, out_lse,
                          reinterpret_cast<cudaStream_t>(cuda_stream));
}

int psd_select_unmask(const float* conf, const int32_t* tok, const int32_t* node, int32_t n_nodes,
                      int32_t* tokens, int32_t* mask, int32_t B, int32_t M, psd_policy_t p,
                      int32_t* sel, int32_t* n_sel, int32_t* sel_pos, void* cuda_stream) {
    if (!conf || !tok || !tokens || !mask || !sel || !n_sel || !sel_pos) return PSD_ERR_NULL;
    if (check_block_shape(B, M) || n_nodes < 1 || n_nodes > PSD_MAX_DEPTH) return PSD_ERR_SHAPE;
    if (int e = check_policy(p)) return e;
    return launch_select(conf, tok, node, n_nodes, tokens, mask, B, M, p, sel, n_sel, sel_pos,
                         reinterpret_cast<cudaStream_t>(cuda_stream));
}

int psd_build_drafts(const float* conf, const int32_t* tok, const int32_t* node, int32_t n_nodes,
                     const int32_t* tokens, const int32_t* mask, int32_t B, int32_t M, psd_policy_t p,
                     int32_t* sigma, int32_t* n_fill, int32_t* draft_tokens, int32_t* draft_mask,
                     void* cuda_stream) {
    if (!conf || !tok || !tokens || !mask || !sigma || !n_fill || !draft_tokens || !draft_mask) return PSD_ERR_NULL;
    if (check_block_shape(B, M) || n_nodes < 1 || n_nodes > PSD_MAX_DEPTH) return PSD_ERR_SHAPE;
    if (int e = check_policy(p)) return e;
    return launch_build(conf, tok, node, n_nodes, tokens, mask, B, M, p, sigma, n_fill, draft_tokens, draft_mask,
                        reinterpret_cast<cudaStream_t>(cuda_stream));
}

int psd_verify_accept(const int32_t* tokV, const float* confV, const int32_t* sigma, const int32_t* n_fill,
                      const int32_t* draft_tokens, const int32_t* draft_mask, int32_t B, int32_t M, psd_policy_t p,
                      int32_t* tokens, int32_t* mask, int32_t* k_star, int32_t* n_spec_accepted,
                      int32_t* n_committed, int32_t* accepted, void* cuda_stream) {
    if (!tokV || !confV || !sigma || !n_fill || !draft_tokens || !draft_mask || !tokens || !mask || !k_star ||
        !n_spec_accepted || !n_committed)
        return PSD_ERR_NULL;
    if (check_block_shape(B, M)) return PSD_ERR_SHAPE;
    if (int e = check_policy(p)) return e;
    return launch_accept(tokV, confV, sigma, n_fill, draft_tokens, draft_mask, B, M, p, tokens, mask, k_star,
                         n_spec_accepted, n_committed, accepted, reinterpret_cast<cudaStream_t>(cuda_stream));
}

static int check_step_io(const psd_step_io_t* io) {
    if (!io) return PSD_ERR_NULL;
    if (!io->hidden_bf16 || !io->w_lm_bf16 || !io->sigma || !io->n_fill || !io->draft_tokens || !io->draft_mask ||
        !io->tokV || !io->confV || !io->tokens || !io->mask || !io->k_star || !io->n_spec_accepted ||
        !io->n_committed || !io->sel || !io->n_sel || !io->sel_pos)
        return PSD_ERR_NULL;
    return PSD_OK;
}

// One step for the chain of p.depth nodes (g == NULL) or for the draft graph g.
static int step_impl(const psd_step_io_t* io, int32_t B, int32_t M, int32_t H, int32_t V, psd_policy_t p,
                     const psd_dag_t* g, void* workspace, size_t workspace_bytes, int32_t* status_dev,
                     void* cuda_stream) {
    if (int e = check_step_io(io)) return e;
    if (check_block_shape(B, M)) return PSD_ERR_SHAPE;
    if (g) {
        if (g->n_nodes < 1 || g->n_nodes > PSD_MAX_DAG_NODES) return PSD_ERR_SHAPE;
        p.depth = g->n_nodes;
    }
    if (int e = check_policy(p)) return e;
    const int D = p.depth;
    if ((long long)B * D * M > 2147483647ll) return PSD_ERR_SHAPE;
    const int n_rows = B * D * M;
    if (!conf_shape_ok(n_rows, H, V)) return PSD_ERR_SHAPE;
    if (!workspace) return PSD_ERR_NULL;
    if (!aligned(io->hidden_bf16, 16) || !aligned(io->w_lm_bf16, 16) || !aligned(workspace, 256) ||
        !aligned(status_dev, 4))
        return PSD_ERR_ALIGN;
    const bool compact = psd_compact_rows_enabled(n_rows) != 0;
    if (workspace_bytes < (compact ? psd_compact_workspace_bytes(n_rows, H, V) : psd_workspace_bytes(n_rows, H, V)))
        return PSD_ERR_WORKSPACE;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
    Partials part = carve_partials(workspace, n_rows, V);
    const void* hidden = io->hidden_bf16;
    const int32_t* pos = nullptr;
    const int32_t* n_rows_dev = nullptr;
    if (compact) {
        // Only the rows of slots still masked in their draft are scored (Stage 3 needs no others): list
        // them, copy their hidden states into a dense buffer, and let the fused kernel read the count
        // from the device, so the step still needs no host synchronisation.
        CompactSpace cs = carve_compact(workspace, n_rows, H, V);
        if (int e = launch_list_rows(io->draft_mask, n_rows, cs.row_ids, cs.pos, cs.count, st)) return e;
        if (int e = launch_gather_rows(hidden, cs.row_ids, cs.count, 0, n_rows, H, cs.hidden, st)) return e;
        hidden = cs.hidden;
        pos = cs.pos;
        n_rows_dev = cs.count;
    }
    // Two launches: the fused LM-head + confidence kernel, then one kernel per sequence block that
    // merges the split-V partials and runs acceptance, the policy on node k* and the next drafts.
    const bool timed = t_ev_start && t_ev_stop;
    if (timed && cudaEventRecord(t_ev_start, st) != cudaSuccess) return PSD_ERR_CUDA;
    SplitPlan plan;
    const int rc = launch_confidence(hidden, io->w_lm_bf16, n_rows, H, V, part, status_dev, st, &plan, n_rows_dev);
    if (timed) {
        cudaError_t ce = cudaEventRecord(t_ev_stop, st);
        t_ev_start = t_ev_stop = nullptr;
        if (ce != cudaSuccess) return PSD_ERR_CUDA;
    }
    if (rc < 0) return rc;
    if (!g)
        return launch_step_tail(part, plan, n_rows, B, M, p, io->tokV, io->confV, io->sigma, io->n_fill,
                                io->draft_tokens, io->draft_mask, io->tokens, io->mask, io->k_star,
                                io->n_spec_accepted, io->n_committed, io->sel, io->n_sel, io->sel_pos, st, pos, status_dev);
    // draft graph: the same stages as separate launches (merge, acceptance over the graph, policy on
    // node k*, next drafts of the graph)
    if (int e = launch_combine(part, plan, n_rows, io->tokV, io->confV, nullptr, st, pos, nullptr, 0, status_dev)) return e;
    if (int e = psd_verify_accept_dag(io->tokV, io->confV, io->sigma, io->draft_tokens, io->draft_mask, B, M, p, g,
                                      io->tokens, io->mask, io->k_star, io->n_spec_accepted, io->n_committed,
                                      nullptr, cuda_stream))
        return e;
    if (int e = launch_select(io->confV, io->tokV, io->k_star, D, io->tokens, io->mask, B, M, p, io->sel, io->n_sel,
                              io->sel_pos, st))
        return e;
    return psd_build_drafts_dag(io->confV, io->tokV, io->k_star, D, io->tokens, io->mask, B, M, p, g, io->sigma,
                                io->n_fill, io->draft_tokens, io->draft_mask, cuda_stream);
}

int psd_step(const psd_step_io_t* io, int32_t B, int32_t M, int32_t H, int32_t V, psd_policy_t p,
             void* workspace, size_t workspace_bytes, int32_t* status_dev, void* cuda_stream) {
    return step_impl(io, B, M, H, V, p, nullptr, workspace, workspace_bytes, status_dev, cuda_stream);
}

int psd_step_dag(const psd_step_io_t* io, int32_t B, int32_t M, int32_t H, int32_t V, psd_policy_t p,
                 const psd_dag_t* g, void* workspace, size_t workspace_bytes, int32_t* status_dev,
                 void* cuda_stream) {
    if (!g) return PSD_ERR_NULL;
    return step_impl(io, B, M, H, V, p, g, workspace, workspace_bytes, status_dev, cuda_stream);
}

// Device staging layout of psd_step_host, in order; every piece 256-byte aligned.
namespace {
struct Staging {
    size_t hidden, sigma, n_fill, draft_tokens, draft_mask, tokV, confV, tokens, mask, k_star, n_spec, n_comm,
        sel, n_sel, sel_pos, status, workspace, total;
};
Staging staging_layout(int B, int M, int H, int V, int D) {
    Staging s;
    size_t o = 0;
    auto take = [&](size_t bytes) { size_t at = o; o += round_up(bytes, 256); return at; };
    const size_t R = (size_t)B * D * M, BM = (size_t)B * M;
    s.hidden = take(R * H * 2);
    s.sigma = take(BM * 4);
    s.n_fill = take((size_t)B * D * 4);
    s.draft_tokens = take(R * 4);
    s.draft_mask = take(R * 4);
    s.tokV = take(R * 4);
    s.confV = take(R * 4);
    s.tokens = take(BM * 4);
    s.mask = take(BM * 4);
    s.k_star = take((size_t)B * 4);
    s.n_spec = take((size_t)B * 4);
    s.n_comm = take((size_t)B * 4);
    s.sel = take(BM * 4);
    s.n_sel = take((size_t)B * 4);
    s.sel_pos = take(BM * 4);
    s.status = take(4);
    s.workspace = take(psd_compact_workspace_bytes((int)R, H, V));   // also enough when row compaction is on
    s.total = o;
    return s;
}
}  // namespace

size_t psd_step_host_block(int32_t B, int32_t M, int32_t D, size_t* offsets) {
    if (check_block_shape(B, M) || D < 1 || D > PSD_MAX_DEPTH || (long long)B * D * M > 2147483647ll) return 0;
    // H and V only size pieces outside [sigma, status]: any valid pair gives the same offsets in between
    const Staging s = staging_layout(B, M, 64, 1, D);
    const size_t at[15] = {s.sigma, s.n_fill, s.draft_tokens, s.draft_mask, s.tokV, s.confV, s.tokens, s.mask,
                           s.k_star, s.n_spec, s.n_comm, s.sel, s.n_sel, s.sel_pos, s.status};
    if (offsets)
        for (int i = 0; i < 15; ++i) offsets[i] = at[i] - s.sigma;
    return s.status + 256 - s.sigma;
}

size_t psd_step_host_bytes(int32_t B, int32_t M, int32_t H, int32_t V, int32_t D) {
    if (check_block_shape(B, M) || D < 1 || D > PSD_MAX_DEPTH || (long long)B * D * M > 2147483647ll) return 0;
    if (!conf_shape_ok(B * D * M, H, V)) return 0;
    return staging_layout(B, M, H, V, D).total;
}

// One internal stream and two events per device for psd_step_host's overlapped copies, created on the
// first call that needs them and kept until the process exits (host-side objects, no device memory).
namespace {
struct CopyLane {
    cudaStream_t stream = nullptr;
    cudaEvent_t begin = nullptr, chunk[2] = {nullptr, nullptr};
    bool ready = false;
    std::mutex in_use;   // one call at a time records and waits on the lane's events
};
std::mutex g_lane_mu;
CopyLane g_lanes[64];

CopyLane* copy_lane() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    std::lock_guard<std::mutex> lock(g_lane_mu);
    CopyLane& l = g_lanes[dev];
    if (!l.ready) {
        if (cudaStreamCreateWithFlags(&l.stream, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
        if (cudaEventCreateWithFlags(&l.begin, cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&l.chunk[0], cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&l.chunk[1], cudaEventDisableTiming) != cudaSuccess)
            return nullptr;
        l.ready = true;
    }
    return &l;
}

// The step on blocks [b0, b1) of a batch: every array of io advanced to block b0.
psd_step_io_t blocks_from(const psd_step_io_t& io, int b0, int M, int D, int H) {
    psd_step_io_t c = io;
    const size_t bm = (size_t)b0 * M, bd = (size_t)b0 * D, bdm = (size_t)b0 * D * M;
    c.hidden_bf16 = reinterpret_cast<const unsigned char*>(io.hidden_bf16) + bdm * H * 2;
    c.sigma += bm; c.n_fill += bd; c.draft_tokens += bdm; c.draft_mask += bdm;
    c.tokV += bdm; c.confV += bdm; c.tokens += bm; c.mask += bm;
    c.k_star += b0; c.n_spec_accepted += b0; c.n_committed += b0;
    c.sel += bm; c.n_sel += b0; c.sel_pos += bm;
    return c;
}
}  // namespace

int psd_step_host(const psd_step_io_t* io, int32_t B, int32_t M, int32_t H, int32_t V, psd_policy_t p,
                  void* staging, size_t staging_bytes, int32_t* status_host, void* cuda_stream) {
    if (int e = check_step_io(io)) return e;
    if (!staging) return PSD_ERR_NULL;
    if (check_block_shape(B, M)) return PSD_ERR_SHAPE;
    if (int e = check_policy(p)) return e;
    const int D = p.depth;
    const size_t need = psd_step_host_bytes(B, M, H, V, D);
    if (need == 0) return PSD_ERR_SHAPE;
    if (!aligned(staging, 256)) return PSD_ERR_ALIGN;
    if (staging_bytes < need) return PSD_ERR_WORKSPACE;
    const Staging s = staging_layout(B, M, H, V, D);
    unsigned char* d = reinterpret_cast<unsigned char*>(staging);
    cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
    const size_t R = (size_t)B * D * M, BM = (size_t)B * M;
    bool ok = true;
    // One block: when the caller's arrays sit in host memory exactly as psd_step_host_block lays them
    // out, the draft state goes up in one copy and every output comes back in one.
    unsigned char* hb = reinterpret_cast<unsigned char*>(io->sigma);
    auto at = [&](const void* ptr, size_t off) { return reinterpret_cast<const unsigned char*>(ptr) == hb + (off - s.sigma); };
    const bool one_block = at(io->n_fill, s.n_fill) && at(io->draft_tokens, s.draft_tokens) &&
                           at(io->draft_mask, s.draft_mask) && at(io->tokV, s.tokV) && at(io->confV, s.confV) &&
                           at(io->tokens, s.tokens) && at(io->mask, s.mask) && at(io->k_star, s.k_star) &&
                           at(io->n_spec_accepted, s.n_spec) && at(io->n_committed, s.n_comm) && at(io->sel, s.sel) &&
                           at(io->n_sel, s.n_sel) && at(io->sel_pos, s.sel_pos);
    auto h2d = [&](size_t off, const void* src, size_t bytes, cudaStream_t on) {
        ok = ok && cudaMemcpyAsync(d + off, src, bytes, cudaMemcpyHostToDevice, on) == cudaSuccess;
    };
    auto d2h = [&](void* dst, size_t off, size_t bytes) {
        ok = ok && cudaMemcpyAsync(dst, d + off, bytes, cudaMemcpyDeviceToHost, st) == cudaSuccess;
    };

    // A large batch goes up in two pieces so that the second copy runs under the first piece's kernels:
    // blocks are independent, so the step on blocks [0, b_cut) and on [b_cut, B) is two psd_step calls.
    // The first piece is kept small (only its copy is exposed) but not so small that its kernel runs in
    // the inefficient range: a quarter of the rows, between 512 and 1024 rows, in whole blocks.
    int b_cut = B;
    const size_t rows_per_block = (size_t)D * M;
    if (R >= 2048 && B >= 2) {
        size_t first_rows = R / 4;
        if (first_rows < 512) first_rows = 512;
        if (first_rows > 1024) first_rows = 1024;
        b_cut = (int)((first_rows + rows_per_block - 1) / rows_per_block);
        if (b_cut >= B) b_cut = B;
    }
    CopyLane* lane = b_cut < B ? copy_lane() : nullptr;
    if (b_cut < B && !lane) b_cut = B;     // no internal stream: fall back to one piece
    std::unique_lock<std::mutex> lane_lock;
    if (lane) lane_lock = std::unique_lock<std::mutex>(lane->in_use);

    // the small arrays first (inputs; in the one-block form the whole block, whose status word the
    // host zeroes here, so the device word needs no separate clearing)
    if (one_block) {
        *reinterpret_cast<int32_t*>(hb + (s.status - s.sigma)) = 0;
        h2d(s.sigma, io->sigma, s.status + 4 - s.sigma, st);
    } else {
        h2d(s.sigma, io->sigma, BM * 4, st);
        h2d(s.n_fill, io->n_fill, (size_t)B * D * 4, st);
        h2d(s.draft_tokens, io->draft_tokens, R * 4, st);
        h2d(s.draft_mask, io->draft_mask, R * 4, st);
        ok = ok && cudaMemsetAsync(d + s.status, 0, 4, st) == cudaSuccess;
    }
    const unsigned char* hid = reinterpret_cast<const unsigned char*>(io->hidden_bf16);
    const size_t cut_bytes = (size_t)b_cut * rows_per_block * H * 2;
    if (b_cut == B) {
        h2d(s.hidden, hid, R * H * 2, st);
    } else {
        // the internal stream starts after everything already queued on the caller's stream (an earlier
        // call may still be reading the staging area), then carries both copies in order
        ok = ok && cudaEventRecord(lane->begin, st) == cudaSuccess;
        ok = ok && cudaStreamWaitEvent(lane->stream, lane->begin, 0) == cudaSuccess;
        h2d(s.hidden, hid, cut_bytes, lane->stream);
        ok = ok && cudaEventRecord(lane->chunk[0], lane->stream) == cudaSuccess;
        h2d(s.hidden + cut_bytes, hid + cut_bytes, R * H * 2 - cut_bytes, lane->stream);
        ok = ok && cudaEventRecord(lane->chunk[1], lane->stream) == cudaSuccess;
    }
    if (!ok) return PSD_ERR_CUDA;

    psd_step_io_t dev;
    dev.hidden_bf16 = d + s.hidden;
    dev.w_lm_bf16 = io->w_lm_bf16;
    dev.sigma = reinterpret_cast<int32_t*>(d + s.sigma);
    dev.n_fill = reinterpret_cast<int32_t*>(d + s.n_fill);
    dev.draft_tokens = reinterpret_cast<int32_t*>(d + s.draft_tokens);
    dev.draft_mask = reinterpret_cast<int32_t*>(d + s.draft_mask);
    dev.tokV = reinterpret_cast<int32_t*>(d + s.tokV);
    dev.confV = reinterpret_cast<float*>(d + s.confV);
    dev.tokens = reinterpret_cast<int32_t*>(d + s.tokens);
    dev.mask = reinterpret_cast<int32_t*>(d + s.mask);
    dev.k_star = reinterpret_cast<int32_t*>(d + s.k_star);
    dev.n_spec_accepted = reinterpret_cast<int32_t*>(d + s.n_spec);
    dev.n_committed = reinterpret_cast<int32_t*>(d + s.n_comm);
    dev.sel = reinterpret_cast<int32_t*>(d + s.sel);
    dev.n_sel = reinterpret_cast<int32_t*>(d + s.n_sel);
    dev.sel_pos = reinterpret_cast<int32_t*>(d + s.sel_pos);
    int32_t* status_dev = reinterpret_cast<int32_t*>(d + s.status);
    if (b_cut == B) {
        if (int e = psd_step(&dev, B, M, H, V, p, d + s.workspace, need - s.workspace, status_dev, cuda_stream)) return e;
    } else {
        // the second piece reuses the workspace: stream order puts it after the first piece's last kernel
        if (cudaStreamWaitEvent(st, lane->chunk[0], 0) != cudaSuccess) return PSD_ERR_CUDA;
        if (int e = psd_step(&dev, b_cut, M, H, V, p, d + s.workspace, need - s.workspace, status_dev, cuda_stream)) return e;
        if (cudaStreamWaitEvent(st, lane->chunk[1], 0) != cudaSuccess) return PSD_ERR_CUDA;
        const psd_step_io_t rest = blocks_from(dev, b_cut, M, D, H);
        if (int e = psd_step(&rest, B - b_cut, M, H, V, p, d + s.workspace, need - s.workspace, status_dev, cuda_stream)) return e;
        lane_lock.unlock();
    }

    if (one_block) {
        // [sigma .. status]: the status word lands in the caller's block, at the offset the layout gives it
        d2h(io->sigma, s.sigma, s.status + 4 - s.sigma);
        ok = ok && cudaStreamSynchronize(st) == cudaSuccess;
        if (!ok) return PSD_ERR_CUDA;
        if (status_host) *status_host = *reinterpret_cast<const int32_t*>(hb + (s.status - s.sigma));
        return PSD_OK;
    }
    d2h(io->sigma, s.sigma, BM * 4);
    d2h(io->n_fill, s.n_fill, (size_t)B * D * 4);
    d2h(io->draft_tokens, s.draft_tokens, R * 4);
    d2h(io->draft_mask, s.draft_mask, R * 4);
    d2h(io->tokV, s.tokV, R * 4);
    d2h(io->confV, s.confV, R * 4);
    d2h(io->tokens, s.tokens, BM * 4);
    d2h(io->mask, s.mask, BM * 4);
    d2h(io->k_star, s.k_star, (size_t)B * 4);
    d2h(io->n_spec_accepted, s.n_spec, (size_t)B * 4);
    d2h(io->n_committed, s.n_comm, (size_t)B * 4);
    d2h(io->sel, s.sel, BM * 4);
    d2h(io->n_sel, s.n_sel, (size_t)B * 4);
    d2h(io->sel_pos, s.sel_pos, BM * 4);
    int32_t status = 0;
    ok = ok && cudaMemcpyAsync(&status, d + s.status, 4, cudaMemcpyDeviceToHost, st) == cudaSuccess;
    ok = ok && cudaStreamSynchronize(st) == cudaSuccess;
    if (!ok) return PSD_ERR_CUDA;
    if (status_host) *status_host = status;
    return PSD_OK;
}

}  // extern "C"
