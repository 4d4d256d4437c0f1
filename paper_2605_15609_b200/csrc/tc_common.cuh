// Device and host helpers shared by the tensor-core kernels of libpsd_b200 (single-CTA and CTA-pair
// versions of the fused LM-head + confidence kernel): mbarrier, TMA and tcgen05 wrappers, the
// running (max, sum-exp, argmax) fold, tensor-map construction.  Everything is internal linkage.
#pragma once
#include <atomic>
#include <cuda.h>
#include <cuda_bf16.h>
#include "psd_internal.cuh"

namespace psd {
namespace {


constexpr int BLOCK_M = 128;       // rows per tile (TMEM lanes)
constexpr int BLOCK_N = 256;       // widest vocabulary tile (TMEM columns per accumulator)
constexpr int BLOCK_K = 64;        // bf16 elements per K-slice = one 128-byte swizzle row
constexpr int UMMA_K = 16;
#ifndef PSD_STAGES
#define PSD_STAGES 4
#endif
constexpr int STAGES = PSD_STAGES;   // depth of the shared-memory ring (48 KB per stage)
constexpr int A_BYTES = BLOCK_M * BLOCK_K * 2;   // 16 KB
constexpr int B_BYTES = BLOCK_N * BLOCK_K * 2;   // 32 KB
constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int TMEM_COLS = 2 * BLOCK_N;           // two accumulators
constexpr int NUM_THREADS = 192;                 // warp 0: TMA, warp 1: MMA + TMEM owner, warps 2-5: epilogue
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 /* alignment slack */ + 256 /* barriers */;
constexpr long long WAIT_LIMIT_CYCLES = 4000000000ll;   // about 2 s at B200 clocks: limit of the waits that drain a CTA's
                                                        // own asynchronous work when it gives up, and the default
                                                        // limit of every other wait (TileGeometry::wait_limit)

struct TileGeometry {
    int n_mt;        // row tiles (of 128 rows for the single-CTA kernel, of 256 rows for CTA pairs)
    int n_vt;        // vocabulary tiles
    int unit;        // columns per unit of tile width: 16, or 32 for CTA pairs (each CTA holds half a tile)
    int base_units;  // every vocabulary tile has base_units or base_units + 1 units
    int rem;         // the first `rem` vocabulary tiles have base_units + 1
    int carry;       // 1: carried partials (see SplitPlan): bands of `band` row tiles, each CTA keeps one running
                     //    triple per row of every row tile it meets in a band and writes it at the band's end;
                     //    0: one triple per (row, vocabulary tile), tile order as decode_tile says
    int band;        // tiles per band of the tile order (see decode_tile, TileCursor)
    int row_bands;   // 0: bands of vocabulary tiles, 1: bands of row tiles
    long long wait_limit;   // clock cycles after which a wait on a barrier gives up (PSD_TUNE_WAIT_LIMIT)
    int stall_test;         // 1: self-test of the give-up path, see PSD_TUNE_SELFTEST_STALL
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// ---- mbarrier ---------------------------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}

// What a wait needs to know to give up: the CTA's abort flag (every role polls it), where to report,
// how long to wait, and for a CTA pair the partner's abort flag (an address in the cluster's shared
// window, 0 for none) so that the two CTAs give up together.
struct WaitCtx {
    volatile int* abort_flag;
    int32_t* status_dev;
    long long limit;
    uint32_t partner_flag;
};
__device__ __forceinline__ void raise_abort(const WaitCtx& w) {
    *w.abort_flag = 1;
    if (w.partner_flag)
        asm volatile("st.relaxed.cluster.shared::cluster.u32 [%0], %1;" ::"r"(w.partner_flag), "r"(1u) : "memory");
    // a count of non-finite rows left by an earlier call gives way to the error code
    if (w.status_dev) atomicMin(w.status_dev, (int)PSD_ERR_TIMEOUT);
}

// Bounded wait.  Returns false if the CTA is aborting (this wait or another one ran out).
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, const WaitCtx& w) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    for (;;) {
        for (int i = 0; i < 256; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (*w.abort_flag) return false;
        if (clock64() - t0 > w.limit) {
            raise_abort(w);
            return false;
        }
    }
}

// ---- TMA --------------------------------------------------------------------------------------
__device__ __forceinline__ void tma_load_2d(void* smem_dst, const CUtensorMap* map, uint64_t* bar, int x, int y,
                                            uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
        " [%0], [%1, {%3, %4}], [%2], %5;"
        ::"r"(smem_u32(smem_dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(smem_u32(bar)), "r"(x), "r"(y),
        "l"(policy)
        : "memory");
}
__device__ __forceinline__ void tma_prefetch_desc(const CUtensorMap* map) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(map)) : "memory");
}

// ---- tcgen05 ----------------------------------------------------------------------------------
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Shared-memory operand descriptor: K-major tile of rows x 64 bf16 written by TMA with the 128-byte
// swizzle.  Rows are 128 bytes apart, groups of 8 rows are 1024 bytes apart (stride byte offset);
// the leading byte offset is not used by swizzled K-major layouts.
__device__ __forceinline__ uint64_t umma_smem_desc(uint32_t smem_addr) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3FFFF) >> 4);        // start address, bits [0,14)
    d |= (uint64_t)1 << 16;                             // leading byte offset (unused), bits [16,30)
    d |= (uint64_t)(1024 >> 4) << 32;                   // stride byte offset, bits [32,46)
    d |= (uint64_t)1 << 46;                             // descriptor version for sm_100
    d |= (uint64_t)2 << 61;                             // layout type: 128-byte swizzle
    return d;
}

// Instruction descriptor, kind::f16: D = fp32, A = B = bf16, both K-major, M = 128, N = n.
__device__ __forceinline__ uint32_t umma_idesc(int n) {
    return (1u << 4)            // D format fp32
         | (1u << 7)            // A format bf16
         | (1u << 10)           // B format bf16
         | ((uint32_t)(n >> 3) << 17)
         | ((uint32_t)(BLOCK_M >> 4) << 24);
}

__device__ __forceinline__ void umma_f16(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc,
                                         uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
        : "memory");
}

// Arrives on the mbarrier once every tcgen05.mma issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                 ::"r"(smem_u32(bar)) : "memory");
}

// 32 lanes x 32 consecutive fp32 columns: thread i of the warp receives lane (base lane + i).
__device__ __forceinline__ void tmem_ld_32x32(uint32_t taddr, float (&v)[32]) {
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

__device__ __forceinline__ void tmem_ld_32x16(uint32_t taddr, float (&v)[32]) {
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
#pragma unroll
    for (int i = 16; i < 32; ++i) v[i] = -INFINITY;
}

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ uint64_t l2_policy_evict_first() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ uint64_t l2_policy_evict_last() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ uint64_t l2_policy_evict_normal() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_normal.b64 %0, 1.0;" : "=l"(p));
    return p;
}

// First column and width of vocabulary tile v_tile.
__host__ __device__ __forceinline__ void tile_columns(const TileGeometry& g, int v_tile, int& v0, int& ncols) {
    const int units0 = v_tile < g.rem ? v_tile * (g.base_units + 1)
                                      : g.rem * (g.base_units + 1) + (v_tile - g.rem) * g.base_units;
    v0 = units0 * g.unit;
    ncols = (v_tile < g.rem ? g.base_units + 1 : g.base_units) * g.unit;
}

// Tile t -> (row tile, first vocabulary column, width).  The tile list is cut into bands so that
// one operand stays in L2 while the other streams past it once per band; the SMs work on consecutive
// t at any moment.
//   g.row_bands == 0: bands of g.band vocabulary tiles.  Inside a band the order is (row tile,
//     vocabulary tile) with the vocabulary tile fastest: the band of W is resident, every row tile of
//     `hidden` is fetched once per band.
//   g.row_bands == 1: bands of g.band row tiles.  Inside a band the order is (vocabulary tile, row
//     tile) with the row tile fastest: the band of `hidden` is resident, W is fetched once per band.
__host__ __device__ __forceinline__ void decode_tile(const TileGeometry& g, int t, int& m_tile, int& v_tile, int& v0,
                                            int& ncols) {
    if (g.row_bands) {
        const int per_band = g.band * g.n_vt;
        const int band = t / per_band;
        const int r = t - band * per_band;
        const int height = min(g.band, g.n_mt - band * g.band);   // the last band may be shorter
        v_tile = r / height;
        m_tile = band * g.band + (r - v_tile * height);
    } else {
        const int per_band = g.band * g.n_mt;
        const int band = t / per_band;
        const int r = t - band * per_band;
        const int width = min(g.band, g.n_vt - band * g.band);    // the last band may be narrower
        m_tile = r / width;
        v_tile = band * g.band + (r - m_tile * width);
    }
    tile_columns(g, v_tile, v0, ncols);
}

// The sequence of tiles of one CTA (or CTA pair) `c` out of `G`, the same in every role of the kernel.
//   g.carry == 0: tiles c, c + G, c + 2G, .. of the global list, decoded by decode_tile.
//   g.carry == 1: the row tiles are cut into bands (heights from band_height: g.band, shrunk so that a
//     CTA meets at most kCarryEntries row tiles per band); inside a band the order is (vocabulary tile,
//     row tile) with the row tile fastest, so the band of `hidden` stays in L2 while W streams past it
//     once, and the G CTAs take the band's tiles round-robin starting again from the band's first tile.
//     After a CTA's last tile of a band (also when it had none) the cursor reports the band's end once:
//     that is where the epilogue writes its carried triples.
struct TileCursor {
    enum { DONE = 0, TILE = 1, BAND_END = 2 };
    int c, G, n_mt, n_tiles;
    int t;                    // flat form: next tile
    int m0, h, gcd, r;        // carried form: first row tile and height of the current band, gcd(G, h), next local tile
    // outputs of next()
    int m_tile, v_tile, v0, ncols;
    int end_m0, end_h, end_gcd;   // the band that just ended (BAND_END)

    __host__ __device__ __forceinline__ void begin(const TileGeometry& g, int c_, int G_, int n_mt_) {
        c = c_; G = G_; n_mt = n_mt_;
        n_tiles = n_mt * g.n_vt;
        t = c;
        m0 = 0; r = c;
        h = n_mt > 0 ? band_height(G, g.band, n_mt) : 0;
        gcd = h > 0 ? gcd_int(G, h) : 1;
    }
    __host__ __device__ __forceinline__ int next(const TileGeometry& g) {
        if (!g.carry) {
            if (t >= n_tiles) return DONE;
            decode_tile(g, t, m_tile, v_tile, v0, ncols);
            t += G;
            return TILE;
        }
        if (m0 >= n_mt) return DONE;
        if (r < h * g.n_vt) {
            v_tile = r / h;
            m_tile = m0 + (r - v_tile * h);
            tile_columns(g, v_tile, v0, ncols);
            r += G;
            return TILE;
        }
        end_m0 = m0; end_h = h; end_gcd = gcd;
        m0 += h;
        h = m0 < n_mt ? band_height(G, g.band, n_mt - m0) : 0;
        gcd = h > 0 ? gcd_int(G, h) : 1;
        r = c;
        return BAND_END;
    }
};

// Folds 32 logits (columns col0 .. col0+31 of this thread's row) into the running triple.
// run_m is kept pre-multiplied by log2(e) in run_ml2 so that the exponent is one FMA.
__device__ __forceinline__ void fold_chunk(const float (&x)[32], int col0, float& run_m, float& run_s, int& run_a) {
    constexpr float LOG2E = 1.4426950408889634f;
    float cm = x[0];
#pragma unroll
    for (int j = 1; j < 32; ++j) cm = fmaxf(cm, x[j]);
    if (cm > run_m) {
        int idx = 31;
#pragma unroll
        for (int j = 30; j >= 0; --j) idx = (x[j] == cm) ? j : idx;
        run_a = col0 + idx;
        run_s *= ex2((run_m - cm) * LOG2E);
        run_m = cm;
    }
    const float neg_ml2 = -run_m * LOG2E;
    float acc = 0.f;
#pragma unroll
    for (int j = 0; j < 32; ++j) acc += ex2(fmaf(x[j], LOG2E, neg_ml2));
    run_s += acc;
}

// ---- host side --------------------------------------------------------------------------------

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            p = nullptr;
        return reinterpret_cast<EncodeTiledFn>(p);
    }();
    return fn;
}

// A [rows, H] bf16 row-major matrix seen as a 2-D tensor (inner = H), boxes of 64 x box_rows
// elements, 128-byte swizzle, zeros outside.
bool make_map(CUtensorMap* m, const void* base, int rows, int H, int box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {(cuuint64_t)H, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)H * 2};
    cuuint32_t box[2] = {(cuuint32_t)BLOCK_K, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// SM count of the current device (looked up once per device).
int sm_count() {
    static std::atomic<int> cached[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    int v = cached[dev].load(std::memory_order_relaxed);
    if (v > 0) return v;
    if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) return 148;
    cached[dev].store(v, std::memory_order_relaxed);
    return v;
}

// The opt-in to more than 48 KB of dynamic shared memory is a per-device property of a kernel: set it
// the first time the kernel is launched on each device.
template <typename Kernel>
bool ensure_dynamic_smem(Kernel kernel, int bytes, std::atomic<unsigned long long>& done_mask) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return false;
    if ((done_mask.load(std::memory_order_acquire) >> dev) & 1ull) return true;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess) return false;
    done_mask.fetch_or(1ull << dev, std::memory_order_release);
    return true;
}

// Chooses how many vocabulary tiles to cut: every tile at most 256 wide, and the tile count such
// that the slowest SM (ceil(tiles / SMs) tiles of the widest width, plus a fixed per-tile cost for
// the pipeline refill and the exposed part of the epilogue) finishes as early as possible.
// `workers` = CTAs (or CTA pairs) that walk the tile list, `tile_rows` = rows per row tile, `unit` =
// granularity of a tile's width in columns.
TileGeometry choose_geometry(int n_rows, int V, int workers, int max_vt, int tile_rows, int unit) {
    const int sms = workers;
    TileGeometry g;
    g.n_mt = (n_rows + tile_rows - 1) / tile_rows;
    g.unit = unit;
    const int units = (V + unit - 1) / unit;
    const int per_tile_units = BLOCK_N / unit;
    const int vt_min = (units + per_tile_units - 1) / per_tile_units;
    int vt_max = vt_min + sms;
    if (vt_max > units) vt_max = units;
    if (vt_max > max_vt) vt_max = max_vt;
    if (vt_max < vt_min) vt_max = vt_min;
    const long long per_tile_cost = 24;   // in columns
    // Row tiles that share a vocabulary tile in the tile order (the band height, about: the order is
    // chosen after the geometry); wide tiles come first in the vocabulary, so with several row tiles
    // only the first rounds of a band pay the wide width.
    const int h = g.n_mt < 32 ? g.n_mt : 32;
    long long best = -1;
    int best_vt = vt_min;
    for (int vt = vt_min; vt <= vt_max; ++vt) {
        const long long base = units / vt, rem = units % vt;
        const long long wide = (rem ? base + 1 : base) * unit, narrow = base * unit;
        const long long tiles = (long long)g.n_mt * vt;
        const long long rounds = (tiles + sms - 1) / sms;
        long long cost;
        if (g.n_mt == 1) {
            cost = rounds * (wide + per_tile_cost);
        } else {
            // per band of h row tiles: round j starts at vocabulary tile j * sms / h, wide while that is < rem
            const long long band_rounds = ((long long)h * vt + sms - 1) / sms;
            long long wide_rounds = (rem * h + sms - 1) / sms;
            if (wide_rounds > band_rounds) wide_rounds = band_rounds;
            const long long band_cost = wide_rounds * wide + (band_rounds - wide_rounds) * narrow + band_rounds * per_tile_cost;
            cost = band_cost * ((g.n_mt + h - 1) / h);
        }
        if (best < 0 || cost < best) { best = cost; best_vt = vt; }
    }
    g.n_vt = best_vt;
    g.base_units = units / best_vt;
    g.rem = units % best_vt;
    g.carry = 0;
    g.band = 1;
    g.row_bands = 0;
    g.wait_limit = wait_limit_cycles();
    g.stall_test = selftest_stall();
    return g;
}

// Tile order: which operand a band keeps in L2 and how large the band is.  `budget` = bytes of the
// resident operand per band; `tile_rows` = rows per row tile.  The order with the smaller estimate of
// DRAM traffic wins: vocabulary bands read W once and `hidden` once per band, row bands read
// `hidden` once and W once per band.  `force`: 0 = choose, 1 = vocabulary bands, 2 = row bands.
void choose_order(TileGeometry& g, int n_rows, int H, int V, int tile_rows, long long budget, int force) {
    const double w_bytes = (double)V * H * 2, h_bytes = (double)n_rows * H * 2;
    const long long vt_bytes = (long long)(g.base_units + (g.rem ? 1 : 0)) * g.unit * H * 2;
    const long long mt_bytes = (long long)tile_rows * H * 2;
    long long vb = budget / (vt_bytes > 0 ? vt_bytes : 1);
    long long mb = budget / mt_bytes;
    if (vb < 1) vb = 1;
    if (vb > g.n_vt) vb = g.n_vt;
    if (mb < 1) mb = 1;
    if (mb > g.n_mt) mb = g.n_mt;
    const long long n_vbands = (g.n_vt + vb - 1) / vb, n_mbands = (g.n_mt + mb - 1) / mb;
    mb = (g.n_mt + n_mbands - 1) / n_mbands;     // bands of equal height
    const double cost_vocab = w_bytes + h_bytes * (double)n_vbands;
    const double cost_rows = h_bytes + w_bytes * (double)n_mbands;
    const bool rows = force == 2 || (force != 1 && g.n_mt > 1 && cost_rows < cost_vocab);
    g.row_bands = rows ? 1 : 0;
    g.band = (int)(rows ? mb : vb);
}

}  // namespace
}  // namespace psd
