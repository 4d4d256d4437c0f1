// Fused LM-head + confidence kernel for sm_100a (Sec. 3.1: x^ = argmax_v p(v), c = max_v p(v)).
//
// logits[r, v] = sum_j hidden[r, j] * W[v, j] is a dense bf16 contraction, so it runs on the
// 5th-generation tensor cores: TMA brings 128-byte-swizzled K-slices of `hidden` (128 rows) and of
// `W` (up to 256 vocabulary rows) into a shared-memory ring, one thread issues tcgen05.mma
// (M = 128, N = tile width, K = 16, bf16 x bf16 -> fp32) into one of two TMEM accumulators, and
// four epilogue warps read the finished accumulator straight out of TMEM (one thread = one row) and
// fold its columns into a per-row (max, sum-exp, argmax) triple.  Logits never reach shared or
// global memory.  One triple per (row, vocabulary tile) goes to the workspace; the combine kernel
// merges them.
//
// Persistent CTAs (one per SM) walk a static list of tiles; the vocabulary is cut into tiles whose
// widths are multiples of 16 and differ by at most 16, so that the tile count can be chosen to
// balance the SMs (at 128 rows the kernel is bound by the one pass over W, and an uneven split
// would leave SMs idle).
//
// Every wait in the kernel is bounded: when a wait runs out the CTA records PSD_ERR_TIMEOUT,
// raises a CTA-wide abort flag that all roles poll, drains its own asynchronous work with bounded
// waits, frees its TMEM and returns.
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
constexpr int STAGES = 4;
constexpr int A_BYTES = BLOCK_M * BLOCK_K * 2;   // 16 KB
constexpr int B_BYTES = BLOCK_N * BLOCK_K * 2;   // 32 KB
constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int TMEM_COLS = 2 * BLOCK_N;           // two accumulators
constexpr int NUM_THREADS = 192;                 // warp 0: TMA, warp 1: MMA + TMEM owner, warps 2-5: epilogue
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 /* alignment slack */ + 256 /* barriers */;
constexpr long long WAIT_LIMIT_CYCLES = 4000000000ll;   // about 2 s at B200 clocks

struct TileGeometry {
    int n_mt;        // row tiles
    int n_vt;        // vocabulary tiles
    int base_units;  // every vocabulary tile has base_units or base_units + 1 units of 16 columns
    int rem;         // the first `rem` vocabulary tiles have base_units + 1
    int carry;       // 1: a CTA keeps one running triple per row across all its tiles (single row tile)
                     //    and writes it to split slot blockIdx.x; 0: one triple per (row, vocabulary tile)
    int band;        // vocabulary tiles per band of the tile order (see decode_tile)
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

// Bounded wait.  Returns false if the CTA is aborting (this wait or another one ran out).
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag,
                                          int32_t* status_dev) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    for (;;) {
        for (int i = 0; i < 256; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if (clock64() - t0 > WAIT_LIMIT_CYCLES) {
            *abort_flag = 1;
            if (status_dev) atomicCAS(status_dev, 0, (int)PSD_ERR_TIMEOUT);
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

// Tile t -> (row tile, first vocabulary column, width).  The vocabulary tiles are grouped in bands
// of g.band tiles; inside a band the order is (row tile, vocabulary tile) with the vocabulary tile
// fastest.  The SMs work on consecutive t at any moment, so together they hold one band of W
// (band * tile bytes, sized to stay in L2 while every row tile passes over it) and a few row tiles of
// `hidden`, each of which is fetched once per band.
__device__ __forceinline__ void decode_tile(const TileGeometry& g, int t, int& m_tile, int& v_tile, int& v0,
                                            int& ncols) {
    const int per_band = g.band * g.n_mt;
    const int band = t / per_band;
    const int r = t - band * per_band;
    const int width = min(g.band, g.n_vt - band * g.band);   // the last band may be narrower
    m_tile = r / width;
    v_tile = band * g.band + (r - m_tile * width);
    const int units0 = v_tile < g.rem ? v_tile * (g.base_units + 1)
                                      : g.rem * (g.base_units + 1) + (v_tile - g.rem) * g.base_units;
    v0 = units0 * 16;
    ncols = (v_tile < g.rem ? g.base_units + 1 : g.base_units) * 16;
}

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

__global__ void __launch_bounds__(NUM_THREADS, 1)
confidence_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b_wide,
                     const __grid_constant__ CUtensorMap map_b_narrow, TileGeometry geo, int n_rows, int H, int V,
                     float* __restrict__ pm, float* __restrict__ ps, int32_t* __restrict__ pa,
                     int32_t* status_dev) {
    extern __shared__ unsigned char smem_raw[];
    // 1024-byte alignment: required by the 128-byte swizzle pattern shared by TMA and the MMA descriptors
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                                           ~static_cast<uintptr_t>(1023));
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + STAGES * STAGE_BYTES);
    uint64_t* full_bar = bars;                    // [STAGES] TMA -> MMA
    uint64_t* empty_bar = bars + STAGES;          // [STAGES] MMA -> TMA
    uint64_t* acc_full_bar = bars + 2 * STAGES;   // [2] MMA -> epilogue
    uint64_t* acc_empty_bar = acc_full_bar + 2;   // [2] epilogue -> MMA
    uint64_t* drain_bar = acc_empty_bar + 2;      // [1] used only when aborting
    uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(drain_bar + 1);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_tiles = geo.n_mt * geo.n_vt;
    const int k_blocks = H / BLOCK_K;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(&acc_full_bar[a], 1);
            mbar_init(&acc_empty_bar[a], 4);   // one arrival per epilogue warp
        }
        mbar_init(drain_bar, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0 && lane == 0) {
        tma_prefetch_desc(&map_a);
        tma_prefetch_desc(&map_b_wide);
        tma_prefetch_desc(&map_b_narrow);
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(tmem_holder)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_holder;

    // Programmatic dependent launch: everything above overlapped the tail of the kernel launched
    // before this one; from here on this kernel reads `hidden` and overwrites the workspace, so it
    // waits for that kernel to finish.
    asm volatile("griddepcontrol.wait;" ::: "memory");

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            // W is read once per row tile: with a single row tile it streams through L2, otherwise the
            // row tiles that run side by side share it for a short while; hidden is re-read for every
            // vocabulary tile and should stay resident.
            const uint64_t pol_w = geo.n_mt > 1 ? l2_policy_evict_normal() : l2_policy_evict_first();
            const uint64_t pol_h = l2_policy_evict_last();
            int q = 0;        // K-slices issued so far
            bool ok = true;
            for (int t = blockIdx.x; t < n_tiles && ok; t += gridDim.x) {
                int m_tile, v_tile, v0, ncols;
                decode_tile(geo, t, m_tile, v_tile, v0, ncols);
                const bool wide = v_tile < geo.rem || geo.rem == 0;
                const CUtensorMap* mb = wide ? &map_b_wide : &map_b_narrow;
                const uint32_t bytes = A_BYTES + (uint32_t)ncols * BLOCK_K * 2;
                for (int kb = 0; kb < k_blocks; ++kb, ++q) {
                    const int s = q % STAGES;
                    if (!mbar_wait(&empty_bar[s], ((q / STAGES) & 1) ^ 1, abort_flag, status_dev)) { ok = false; break; }
                    unsigned char* sa = smem + s * STAGE_BYTES;
                    mbar_arrive_expect_tx(&full_bar[s], bytes);
                    tma_load_2d(sa, &map_a, &full_bar[s], kb * BLOCK_K, m_tile * BLOCK_M, pol_h);
                    tma_load_2d(sa + A_BYTES, mb, &full_bar[s], kb * BLOCK_K, v0, pol_w);
                }
            }
            if (!ok) {
                // Aborting: wait (bounded) until the copies already issued have landed, so that no
                // TMA write is still in flight when the CTA exits.  If the MMA warp has not
                // consumed a slice, its barrier phase is still observable here.
                const int first = q > STAGES ? q - STAGES : 0;
                for (int i = first; i < q; ++i) {
                    const long long t0 = clock64();
                    while (!mbar_try_wait(&full_bar[i % STAGES], (i / STAGES) & 1) && clock64() - t0 < WAIT_LIMIT_CYCLES) {}
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            int q = 0, it = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < n_tiles && ok; t += gridDim.x, ++it) {
                int m_tile, v_tile, v0, ncols;
                decode_tile(geo, t, m_tile, v_tile, v0, ncols);
                const int acc = it & 1;
                if (!mbar_wait(&acc_empty_bar[acc], ((it >> 1) & 1) ^ 1, abort_flag, status_dev)) { ok = false; break; }
                tc_fence_after();
                const uint32_t idesc = umma_idesc(ncols);
                const uint32_t tmem_d = tmem_base + (uint32_t)(acc * BLOCK_N);
                for (int kb = 0; kb < k_blocks; ++kb, ++q) {
                    const int s = q % STAGES;
                    if (!mbar_wait(&full_bar[s], (q / STAGES) & 1, abort_flag, status_dev)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t a_addr = smem_u32(smem + s * STAGE_BYTES);
                    const uint64_t da = umma_smem_desc(a_addr);
                    const uint64_t db = umma_smem_desc(a_addr + A_BYTES);
#pragma unroll
                    for (int k = 0; k < BLOCK_K / UMMA_K; ++k) {
                        // advancing K by 16 elements = 32 bytes inside the swizzle row: +2 in 16-byte units
                        umma_f16(tmem_d, da + (uint64_t)(k * 2), db + (uint64_t)(k * 2), idesc, (kb | k) != 0);
                    }
                    umma_commit(&empty_bar[s]);       // the slice can be overwritten once these MMAs are done
                }
                if (ok) umma_commit(&acc_full_bar[acc]);
            }
            if (!ok) {
                // Aborting: make sure no MMA is still writing TMEM before it is freed.
                umma_commit(drain_bar);
                const long long t0 = clock64();
                while (!mbar_try_wait(drain_bar, 0) && clock64() - t0 < WAIT_LIMIT_CYCLES) {}
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2..5)
        // A warp may only touch the 32 TMEM lanes of its own quarter: quarter = warp index mod 4.
        const int quarter = warp & 3;
        const int row_in_tile = quarter * 32 + lane;
        int it = 0;
        bool ok = true;
        float run_m = -INFINITY, run_s = 0.f;
        int run_a = 0;
        for (int t = blockIdx.x; t < n_tiles && ok; t += gridDim.x, ++it) {
            int m_tile, v_tile, v0, ncols;
            decode_tile(geo, t, m_tile, v_tile, v0, ncols);
            const int acc = it & 1;
            if (!mbar_wait(&acc_full_bar[acc], (it >> 1) & 1, abort_flag, status_dev)) { ok = false; break; }
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * BLOCK_N);
            if (!geo.carry) { run_m = -INFINITY; run_s = 0.f; run_a = 0; }
            const bool ragged = v0 + ncols > V;      // only the last vocabulary tile can reach past V
            for (int c = 0; c < ncols; c += 32) {
                float x[32];
                if (ncols - c >= 32) tmem_ld_32x32(taddr + c, x);
                else tmem_ld_32x16(taddr + c, x);
                if (ragged) {
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        if (v0 + c + j >= V) x[j] = -INFINITY;   // columns past V hold zeros, not logits
                }
                fold_chunk(x, v0 + c, run_m, run_s, run_a);
            }
            // all of this warp's TMEM reads are complete (wait::ld inside the loads): hand the accumulator back
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&acc_empty_bar[acc]);
            // A CTA's tiles come in ascending vocabulary order, so a carried triple keeps the lowest
            // index among equal maxima just as the per-tile triples do after the merge.
            const bool last_of_cta = t + (int)gridDim.x >= n_tiles;
            const int row = m_tile * BLOCK_M + row_in_tile;
            if (row < n_rows && (!geo.carry || last_of_cta)) {
                const size_t o = (size_t)(geo.carry ? (int)blockIdx.x : v_tile) * n_rows + row;
                pm[o] = run_m;
                ps[o] = run_s;
                pa[o] = run_a;
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    // This CTA's tiles are done: once every CTA is here the kernel launched next may become resident
    // and run its set-up (it still waits for this whole grid before it reads the partial triples).
    // Releasing it any earlier would park its thread blocks on the SMs beside the CTAs still working.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
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

int sm_count() {
    static int n = [] {
        int dev = 0, v = 0;
        if (cudaGetDevice(&dev) != cudaSuccess) return 148;
        if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) return 148;
        return v;
    }();
    return n;
}

// Chooses how many vocabulary tiles to cut: every tile at most 256 wide, and the tile count such
// that the slowest SM (ceil(tiles / SMs) tiles of the widest width, plus a fixed per-tile cost for
// the pipeline refill and the exposed part of the epilogue) finishes as early as possible.
TileGeometry choose_geometry(int n_rows, int V, int sms, int max_vt) {
    TileGeometry g;
    g.n_mt = (n_rows + BLOCK_M - 1) / BLOCK_M;
    const int units = (V + 15) / 16;
    const int vt_min = (units + 15) / 16;
    int vt_max = vt_min + sms;
    if (vt_max > units) vt_max = units;
    if (vt_max > max_vt) vt_max = max_vt;
    if (vt_max < vt_min) vt_max = vt_min;
    const long long per_tile_cost = 24;   // in columns
    long long best = -1;
    int best_vt = vt_min;
    for (int vt = vt_min; vt <= vt_max; ++vt) {
        const long long width = ((units + vt - 1) / vt) * 16;
        const long long tiles = (long long)g.n_mt * vt;
        const long long rounds = (tiles + sms - 1) / sms;
        const long long cost = rounds * (width + per_tile_cost);
        if (best < 0 || cost < best) { best = cost; best_vt = vt; }
    }
    g.n_vt = best_vt;
    g.base_units = units / best_vt;
    g.rem = units % best_vt;
    g.carry = g.n_mt == 1 ? 1 : 0;
    return g;
}

std::atomic<int> g_band_bytes{16 << 20};

// Band width: as many vocabulary tiles as fit the L2 budget for W (at least 1, at most all).
int choose_band(const TileGeometry& g, int H) {
    const long long tile_bytes = (long long)(g.base_units + (g.rem ? 1 : 0)) * 16 * H * 2;
    long long b = g_band_bytes.load() / (tile_bytes > 0 ? tile_bytes : 1);
    if (b < 1) b = 1;
    if (b > g.n_vt) b = g.n_vt;
    return (int)b;
}

}  // namespace

void set_band_bytes(int bytes) { g_band_bytes.store(bytes); }

int launch_confidence_tc(const void* hidden, const void* w, int n_rows, int H, int V, Partials part,
                         int32_t* status_dev, cudaStream_t st) {
    static bool attr_set = false;
    if (!attr_set) {
        if (cudaFuncSetAttribute(confidence_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES) !=
            cudaSuccess)
            return PSD_ERR_CUDA;
        attr_set = true;
    }
    const int sms = sm_count();
    TileGeometry g = choose_geometry(n_rows, V, sms, max_splits(V));
    g.band = choose_band(g, H);
    const int wide_rows = (g.rem ? g.base_units + 1 : g.base_units) * 16;
    const int narrow_rows = g.base_units > 0 ? g.base_units * 16 : wide_rows;
    CUtensorMap map_a, map_bw, map_bn;
    if (!make_map(&map_a, hidden, n_rows, H, BLOCK_M) || !make_map(&map_bw, w, V, H, wide_rows) ||
        !make_map(&map_bn, w, V, H, narrow_rows))
        return PSD_ERR_CUDA;
    const int n_tiles = g.n_mt * g.n_vt;
    const int grid = n_tiles < sms ? n_tiles : sms;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(NUM_THREADS);
    cfg.dynamicSmemBytes = SMEM_BYTES;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    // Starting before the kernel ahead has drained hides this kernel's set-up, which matters when the
    // whole pass takes under 200 us (one row tile).  With many row tiles an early start was measured
    // to lengthen the pass by 5-8% (8192 rows), so there the kernel keeps plain stream order.
    attr[0].val.programmaticStreamSerializationAllowed = (pdl_enabled() && g.n_mt == 1) ? 1 : 0;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, confidence_tc_kernel, map_a, map_bw, map_bn, g, n_rows, H, V, part.m,
                                       part.s, part.a, status_dev);
    count_launch();
    if (e != cudaSuccess) return PSD_ERR_CUDA;
    return g.carry ? grid : g.n_vt;   // number of split slots written per row
}

}  // namespace psd
