// Internal declarations shared by the translation units of libpsd_b200 (not part of the ABI).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include <stddef.h>
#include "psd.h"

namespace psd {

// Width (vocabulary entries) of one split of the vocabulary in the tensor-core kernel; the
// workspace is sized for one partial triple per (row, split) at this granularity or coarser.
constexpr int kMinSplitWidth = 128;

// Workspace layout: three arrays [n_split][n_rows] (max, sum-exp, argmax), n_split <= max_splits(V).
inline int max_splits(int V) { return (V + kMinSplitWidth - 1) / kMinSplitWidth; }

struct Partials {
    float* m;      // [n_split][n_rows] running max of the split's logits
    float* s;      // [n_split][n_rows] sum of exp(l - m) over the split
    int32_t* a;    // [n_split][n_rows] lowest vocabulary index attaining m
    size_t cap;    // triples each array holds (checked by the debug build; 0 = not known)
};

inline Partials carve_partials(void* workspace, int n_rows, int V) {
    size_t n = (size_t)max_splits(V) * (size_t)n_rows;
    Partials p;
    p.m = reinterpret_cast<float*>(workspace);
    p.s = p.m + n;
    p.a = reinterpret_cast<int32_t*>(p.s + n);
    p.cap = n;
    return p;
}

// ---- How many partial triples each row has -------------------------------------------------------
// Either the same number for every row (`uniform` > 0), or the carried layout of the single-CTA
// tensor-core kernel: its tile list is cut into bands of row tiles, G CTAs share the tiles of a band
// round-robin, and each CTA carries one running triple per row of every row tile it meets in the band
// and writes it once at the band's end.  With g = gcd(G, band height), CTA c meets the row tiles
// m = (c mod g) + e*g of the band, and a row tile is met by the G/g CTAs of one residue class, which
// write to slots c / g: rows of that band have G/g splits.
constexpr int kTileRows = 128;       // rows per row tile of the single-CTA tensor-core kernel (TMEM lanes)
constexpr int kCarryEntries = 16;    // running triples (row tiles) a CTA can carry per band

struct SplitPlan {
    int uniform;                 // > 0: splits per row, for every row; 0: carried layout (fields below)
    int G;                       // CTAs that walked the tile list
    int hb;                      // nominal band height, in row tiles
    int tile_rows;               // rows per row tile: 128 (single-CTA kernel) or 256 (CTA pairs)
    int n_rows;                  // rows (the capacity when n_rows_dev is given)
    const int32_t* n_rows_dev;   // NULL, or a device word holding how many rows were scored
};
inline SplitPlan uniform_splits(int n) { SplitPlan p = {n, 0, 0, kTileRows, 0, nullptr}; return p; }

__host__ __device__ inline int gcd_int(int a, int b) {
    while (b) { const int t = a % b; a = b; b = t; }
    return a;
}
// Height (row tiles) of the band that begins when `remaining` row tiles are left: at most hb, shrunk
// until a CTA has at most kCarryEntries row tiles to carry.  Heights up to kCarryEntries always qualify.
__host__ __device__ inline int band_height(int G, int hb, int remaining) {
    int h = remaining < hb ? remaining : hb;
    while (h / gcd_int(G, h) > kCarryEntries) --h;
    return h;
}
// Splits of the rows of row tile m under the carried layout with n_mt row tiles in all.
__host__ __device__ inline int carried_splits(int G, int hb, int n_mt, int m) {
    int m0 = 0;
    if (n_mt >= hb) {
        // the leading bands all have the height of a full band: jump over them
        const int h_full = band_height(G, hb, hb);
        const int k_full = (n_mt - hb) / h_full + 1;
        if (m < k_full * h_full) return G / gcd_int(G, h_full);
        m0 = k_full * h_full;
    }
    for (;;) {
        const int h = band_height(G, hb, n_mt - m0);
        if (m < m0 + h || h <= 0) return G / gcd_int(G, h > 0 ? h : 1);
        m0 += h;
    }
}

// Debug build (-DPSD_DEBUG): index and ring-order checks inside the kernels.  A failed check writes
// PSD_ERR_INTERNAL to the status word (when there is one) and the caller skips the access; nothing
// traps.  In the normal build the checks compile to nothing.
#ifdef PSD_DEBUG
__device__ __forceinline__ bool debug_check(bool ok, int32_t* status_dev) {
    if (!ok && status_dev) atomicMin(status_dev, (int)PSD_ERR_INTERNAL);
    return ok;
}
#define PSD_DEBUG_OK(cond, status_dev) (::psd::debug_check((cond), (status_dev)))
#else
#define PSD_DEBUG_OK(cond, status_dev) (true)
#endif

void count_launch(int n = 1);

// 1 when kernels are launched with programmatic stream serialization (a kernel's set-up overlaps the
// tail of the one before it), 0 for plain stream order.
int pdl_enabled();

// confidence_simt.cu: plain CUDA-core kernel. Returns the number of splits written, or < 0.
int launch_confidence_simt(const void* hidden, const void* w, int n_rows, int H, int V,
                           Partials part, cudaStream_t st);

// Tensor-core kernels (tcgen05 + TMA).  Each returns PSD_OK or < 0 (psd_status) and fills *plan with the
// layout of the partial triples it wrote.
// confidence_tc.cu: one CTA per tile of 128 rows; confidence_tc2.cu: a pair of CTAs per tile of 256 rows.
// n_rows_dev: NULL, or a device word holding how many of the n_rows rows actually hold data (the rest
// of the buffer is ignored; n_rows stays the capacity and the stride of the partial arrays).
int launch_confidence_tc1(const void* hidden, const void* w, int n_rows, int H, int V, Partials part,
                          int32_t* status_dev, const int32_t* n_rows_dev, cudaStream_t st, SplitPlan* plan);
int launch_confidence_tc2(const void* hidden, const void* w, int n_rows, int H, int V, Partials part,
                          int32_t* status_dev, const int32_t* n_rows_dev, cudaStream_t st, SplitPlan* plan);
// psd_api.cu: picks the kernel according to psd_set_confidence_impl (the CUDA-core kernel included).
int launch_confidence(const void* hidden, const void* w, int n_rows, int H, int V, Partials part,
                      int32_t* status_dev, cudaStream_t st, SplitPlan* plan, const int32_t* n_rows_dev = nullptr);

long long wait_limit_cycles();   // psd_api.cu: PSD_TUNE_WAIT_LIMIT in clock cycles
int selftest_stall();            // psd_api.cu: PSD_TUNE_SELFTEST_STALL
long long band_bytes();   // psd_api.cu: L2 budget for the operand that a band of the tile order keeps resident
int tile_order();         // psd_api.cu: 0 = choose, 1 = vocabulary bands, 2 = row bands

// compact.cu: ordered list of the rows whose flag is set (row_ids, inverse map pos, count on the device),
// and a gather of those rows of a [*, H] bf16 matrix into a dense buffer.
int launch_list_rows(const int32_t* flags, int n, int32_t* row_ids, int32_t* pos, int32_t* count, cudaStream_t st);
int launch_gather_rows(const void* src, const int32_t* row_ids, const int32_t* count_dev, int count_host, int max_rows,
                       int H, void* dst, cudaStream_t st);

// Extra workspace of the compacted path, after the partial triples: dense hidden rows, row list,
// inverse map, count.
struct CompactSpace {
    void* hidden;       // [n_rows, H] bf16
    int32_t* row_ids;   // [n_rows]
    int32_t* pos;       // [n_rows]
    int32_t* count;     // [1]
};
inline size_t partial_bytes(int n_rows, int V) { return ((size_t)max_splits(V) * (size_t)n_rows * 12 + 255) / 256 * 256; }
inline size_t compact_extra_bytes(int n_rows, int H) {
    return ((size_t)n_rows * H * 2 + 255) / 256 * 256 + ((size_t)n_rows * 8 + 4 + 255) / 256 * 256;
}
inline CompactSpace carve_compact(void* workspace, int n_rows, int H, int V) {
    unsigned char* p = reinterpret_cast<unsigned char*>(workspace) + partial_bytes(n_rows, V);
    CompactSpace c;
    c.hidden = p;
    p += ((size_t)n_rows * H * 2 + 255) / 256 * 256;
    c.row_ids = reinterpret_cast<int32_t*>(p);
    c.pos = c.row_ids + n_rows;
    c.count = c.pos + n_rows;
    return c;
}

// combine.cu: merge n_split partial triples per row.
// pos: NULL, or for every output row the column that holds its partials (-1: the row was not scored
// and its outputs are left alone).
int launch_combine(Partials part, SplitPlan plan, int n_rows,
                   int32_t* out_token, float* out_conf, float* out_lse, cudaStream_t st,
                   const int32_t* pos = nullptr, float* out_max = nullptr, int32_t arg_offset = 0,
                   int32_t* status_dev = nullptr);
// With out_max the kernel writes the merged triple instead: out_max = max, out_conf = sum-exp,
// out_token = argmax + arg_offset.  status_dev: NULL, or the status word that counts non-finite rows.

// policy.cu
int launch_select(const float* conf, const int32_t* tok, const int32_t* node, int n_nodes,
                  int32_t* tokens, int32_t* mask, int B, int M, psd_policy_t p,
                  int32_t* sel, int32_t* n_sel, int32_t* sel_pos, cudaStream_t st);
int launch_build(const float* conf, const int32_t* tok, const int32_t* node, int n_nodes,
                 const int32_t* tokens, const int32_t* mask, int B, int M, psd_policy_t p,
                 int32_t* sigma, int32_t* n_fill, int32_t* draft_tokens, int32_t* draft_mask,
                 cudaStream_t st);
int launch_accept(const int32_t* tokV, const float* confV, const int32_t* sigma, const int32_t* n_fill,
                  const int32_t* draft_tokens, const int32_t* draft_mask, int B, int M, psd_policy_t p,
                  int32_t* tokens, int32_t* mask, int32_t* k_star, int32_t* n_spec, int32_t* n_comm,
                  int32_t* accepted, cudaStream_t st);

// policy.cu: the whole tail of a step in one launch (split-V merge, acceptance, policy, next drafts).
int launch_step_tail(Partials part, SplitPlan plan, int n_rows, int B, int M, psd_policy_t p,
                     int32_t* tokV, float* confV, int32_t* sigma, int32_t* n_fill, int32_t* draft_tokens,
                     int32_t* draft_mask, int32_t* tokens, int32_t* mask, int32_t* k_star, int32_t* n_spec,
                     int32_t* n_comm, int32_t* sel, int32_t* n_sel, int32_t* sel_pos, cudaStream_t st,
                     const int32_t* pos = nullptr, int32_t* status_dev = nullptr);

}  // namespace psd
