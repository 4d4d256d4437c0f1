// Fused LM-head + confidence kernel for sm_100a (Sec. 3.1: x^ = argmax_v p(v), c = max_v p(v)).
//
// logits[r, v] = sum_j hidden[r, j] * W[v, j] is a dense bf16 contraction, so it runs on the
// 5th-generation tensor cores: TMA brings 128-byte-swizzled K-slices of `hidden` (128 rows) and of
// `W` (up to 256 vocabulary rows) into a shared-memory ring, one thread issues tcgen05.mma
// (M = 128, N = tile width, K = 16, bf16 x bf16 -> fp32) into one of two TMEM accumulators, and
// four epilogue warps read the finished accumulator straight out of TMEM (one thread = one row) and
// fold its columns into a per-row (max, sum-exp, argmax) triple.  Logits never reach shared or
// global memory.  Partial triples go to the workspace and the combine pass merges them: with the
// carried layout (the usual case) every CTA keeps one running triple per row of each row tile it meets
// in a band of its tile list, in a small table in shared memory, and writes it once at the band's end
// (a few dozen triples per row, see SplitPlan); otherwise one triple per (row, vocabulary tile).
//
// Persistent CTAs (one per SM) walk a static list of tiles; the vocabulary is cut into tiles whose
// widths are multiples of 16 and differ by at most 16, so that the tile count can be chosen to
// balance the SMs (at 128 rows the kernel is bound by the one pass over W, and an uneven split
// would leave SMs idle).
//
// Every wait in the kernel is bounded: when a wait runs out the CTA records PSD_ERR_TIMEOUT,
// raises a CTA-wide abort flag that all roles poll, drains its own asynchronous work with bounded
// waits, frees its TMEM and returns.
#include <algorithm>
#include <atomic>
#include "tc_common.cuh"

namespace psd {
namespace {

constexpr int BARRIER_BYTES = 256;
constexpr int CARRY_BYTES = kCarryEntries * BLOCK_M * 12;   // carried triples of a CTA (24 KB)
constexpr int SMEM1_BYTES = STAGES * STAGE_BYTES + 1024 /* alignment slack */ + BARRIER_BYTES + CARRY_BYTES;
static_assert(SMEM1_BYTES <= 227 * 1024, "shared memory of the single-CTA kernel");

__global__ void __launch_bounds__(NUM_THREADS, 1)
confidence_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b_wide,
                     const __grid_constant__ CUtensorMap map_b_narrow, TileGeometry geo, int n_rows, int H, int V,
                     float* __restrict__ pm, float* __restrict__ ps, int32_t* __restrict__ pa,
                     int32_t* status_dev, const int32_t* __restrict__ n_rows_dev, size_t part_cap) {
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
    uint64_t* never_bar = drain_bar + 1;          // [1] nothing ever arrives on it (self-test of the give-up path)
    uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(never_bar + 1);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);
#ifdef PSD_DEBUG
    volatile int* ring_tag = abort_flag + 1;   // [stages] the K-slice number the loader put in each stage
#endif
    // carried triples: [kCarryEntries][BLOCK_M] max, then sum-exp, then argmax
    float* carry_m = reinterpret_cast<float*>(smem + STAGES * STAGE_BYTES + BARRIER_BYTES);
    float* carry_s = carry_m + kCarryEntries * BLOCK_M;
    int32_t* carry_a = reinterpret_cast<int32_t*>(carry_s + kCarryEntries * BLOCK_M);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
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
        mbar_init(never_bar, 1);
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

    // The number of rows to score may be known only on the device (rows compacted by the kernel
    // ahead): n_rows then stays the capacity (tensor map, stride of the partial arrays) and the tile
    // list shrinks to the row tiles that hold rows.
    int n_rows_act = n_rows;
    if (n_rows_dev) {
        n_rows_act = min(max(*n_rows_dev, 0), n_rows);
        geo.n_mt = (n_rows_act + BLOCK_M - 1) / BLOCK_M;
    }
    const int n_mt = geo.n_mt;
    const WaitCtx wc = {abort_flag, status_dev, geo.wait_limit, 0u};

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            // One row tile: W streams through L2 once and is marked to leave first; the hidden rows are
            // re-read for every vocabulary tile and stay.  Several row tiles: both operands are re-read
            // from L2 many times within a band, and marking both to stay measured fastest (8192 rows:
            // 6.3 ms against 7.3 ms with the default policy on both, at equal DRAM traffic).
            const uint64_t pol_w = geo.n_mt == 1 ? l2_policy_evict_first() : l2_policy_evict_last();
            const uint64_t pol_h = l2_policy_evict_last();
            int q = 0;        // K-slices issued so far
            bool ok = true;
            TileCursor cur;
            cur.begin(geo, blockIdx.x, gridDim.x, n_mt);
            for (int ev; ok && (ev = cur.next(geo)) != TileCursor::DONE;) {
                if (ev != TileCursor::TILE) continue;
                const int m_tile = cur.m_tile, v_tile = cur.v_tile, v0 = cur.v0, ncols = cur.ncols;
                const bool wide = v_tile < geo.rem || geo.rem == 0;
                const CUtensorMap* mb = wide ? &map_b_wide : &map_b_narrow;
                const uint32_t bytes = A_BYTES + (uint32_t)ncols * BLOCK_K * 2;
                for (int kb = 0; kb < k_blocks; ++kb, ++q) {
                    const int s = q % STAGES;
                    if (!mbar_wait(&empty_bar[s], ((q / STAGES) & 1) ^ 1, wc)) { ok = false; break; }
                    unsigned char* sa = smem + s * STAGE_BYTES;
#ifdef PSD_DEBUG
                    ring_tag[s] = q;
#endif
                    mbar_arrive_expect_tx(&full_bar[s], bytes);
                    tma_load_2d(sa, &map_a, &full_bar[s], kb * BLOCK_K, m_tile * BLOCK_M, pol_h);
                    tma_load_2d(sa + A_BYTES, mb, &full_bar[s], kb * BLOCK_K, v0, pol_w);
                    // self-test of the give-up path: a wait that nothing will ever satisfy, one slice in flight
                    if (geo.stall_test && q == 0 && !mbar_wait(never_bar, 0, wc)) { ok = false; ++q; break; }
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
            TileCursor cur;
            cur.begin(geo, blockIdx.x, gridDim.x, n_mt);
            for (int ev; ok && (ev = cur.next(geo)) != TileCursor::DONE;) {
                if (ev != TileCursor::TILE) continue;
                const int acc = it & 1;
                if (!mbar_wait(&acc_empty_bar[acc], ((it >> 1) & 1) ^ 1, wc)) { ok = false; break; }
                tc_fence_after();
                const uint32_t idesc = umma_idesc(cur.ncols);
                const uint32_t tmem_d = tmem_base + (uint32_t)(acc * BLOCK_N);
                for (int kb = 0; kb < k_blocks; ++kb, ++q) {
                    const int s = q % STAGES;
                    if (!mbar_wait(&full_bar[s], (q / STAGES) & 1, wc)) { ok = false; break; }
                    tc_fence_after();
#ifdef PSD_DEBUG
                    PSD_DEBUG_OK(ring_tag[s] == q, status_dev);   // the stage holds the slice this MMA expects
#endif
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
                ++it;
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
        // carried layout: this thread's entries of the table start neutral (no logit seen)
        auto reset_carry = [&]() {
#pragma unroll
            for (int e = 0; e < kCarryEntries; ++e) {
                carry_m[e * BLOCK_M + row_in_tile] = -INFINITY;
                carry_s[e * BLOCK_M + row_in_tile] = 0.f;
                carry_a[e * BLOCK_M + row_in_tile] = 0;
            }
        };
        if (geo.carry) reset_carry();
        TileCursor cur;
        cur.begin(geo, blockIdx.x, gridDim.x, n_mt);
        for (int ev; ok && (ev = cur.next(geo)) != TileCursor::DONE;) {
            if (ev == TileCursor::BAND_END) {
                // The band is over for this CTA: write the triples it carried, one per row of every row tile
                // of its residue class (those it never reached stay neutral), to its slot of those rows.
                const int entries = cur.end_h / cur.end_gcd;
                const int slot = (int)blockIdx.x / cur.end_gcd, base = (int)blockIdx.x % cur.end_gcd;
                for (int e = 0; e < entries; ++e) {
                    const int row = (cur.end_m0 + base + e * cur.end_gcd) * BLOCK_M + row_in_tile;
                    if (row < n_rows_act && PSD_DEBUG_OK((size_t)slot * n_rows + row < part_cap && e < kCarryEntries, status_dev)) {
                        const size_t o = (size_t)slot * n_rows + row;
                        pm[o] = carry_m[e * BLOCK_M + row_in_tile];
                        ps[o] = carry_s[e * BLOCK_M + row_in_tile];
                        pa[o] = carry_a[e * BLOCK_M + row_in_tile];
                    }
                }
                reset_carry();
                continue;
            }
            const int m_tile = cur.m_tile, v_tile = cur.v_tile, v0 = cur.v0, ncols = cur.ncols;
            const int acc = it & 1;
            if (!mbar_wait(&acc_full_bar[acc], (it >> 1) & 1, wc)) { ok = false; break; }
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * BLOCK_N);
            // A CTA meets the tiles of one row tile in ascending vocabulary order, so a carried triple keeps
            // the lowest index among equal maxima just as per-tile triples do after the merge.
            const int entry = geo.carry ? ((m_tile - cur.m0) / cur.gcd) * BLOCK_M + row_in_tile : 0;
            if (!PSD_DEBUG_OK(m_tile >= 0 && m_tile < n_mt && v0 >= 0 && v0 < V && ncols > 0 && ncols <= BLOCK_N &&
                                  entry >= 0 && entry < kCarryEntries * BLOCK_M, status_dev)) { ok = false; break; }
            float run_m = -INFINITY, run_s = 0.f;
            int run_a = 0;
            if (geo.carry) { run_m = carry_m[entry]; run_s = carry_s[entry]; run_a = carry_a[entry]; }
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
            if (geo.carry) {
                carry_m[entry] = run_m; carry_s[entry] = run_s; carry_a[entry] = run_a;
            } else {
                const int row = m_tile * BLOCK_M + row_in_tile;
                if (row < n_rows_act && PSD_DEBUG_OK((size_t)v_tile * n_rows + row < part_cap, status_dev)) {
                    const size_t o = (size_t)v_tile * n_rows + row;
                    pm[o] = run_m;
                    ps[o] = run_s;
                    pa[o] = run_a;
                }
            }
            ++it;
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

}  // namespace

int launch_confidence_tc1(const void* hidden, const void* w, int n_rows, int H, int V, Partials part,
                          int32_t* status_dev, const int32_t* n_rows_dev, cudaStream_t st, SplitPlan* plan) {
    static std::atomic<unsigned long long> smem_set{0};
    if (!ensure_dynamic_smem(confidence_tc_kernel, SMEM1_BYTES, smem_set)) return PSD_ERR_CUDA;
    const int sms = sm_count();
    TileGeometry g = choose_geometry(n_rows, V, sms, max_splits(V), BLOCK_M, 16);
    choose_order(g, n_rows, H, V, BLOCK_M, band_bytes(), tile_order());
    if (g.n_mt == 1) { g.row_bands = 1; g.band = 1; }   // one row tile: ascending vocabulary order either way
    const int wide_rows = (g.rem ? g.base_units + 1 : g.base_units) * 16;
    const int narrow_rows = g.base_units > 0 ? g.base_units * 16 : wide_rows;
    CUtensorMap map_a, map_bw, map_bn;
    if (!make_map(&map_a, hidden, n_rows, H, BLOCK_M) || !make_map(&map_bw, w, V, H, wide_rows) ||
        !make_map(&map_bn, w, V, H, narrow_rows))
        return PSD_ERR_CUDA;
    const int n_tiles = g.n_mt * g.n_vt;
    const int grid = n_tiles < sms ? n_tiles : sms;
    // Carried partials need row bands, and pay only if they leave fewer triples per row than one per
    // vocabulary tile would (which also keeps them inside the workspace, sized for that).  With the row
    // count on the device the band heights are not known here: take the worst case, one slot per CTA.
    int most_splits = grid;
    if (!n_rows_dev) {
        most_splits = 0;
        for (int m0 = 0; m0 < g.n_mt;) {
            const int h = band_height(grid, g.band, g.n_mt - m0);
            most_splits = std::max(most_splits, grid / gcd_int(grid, h));
            m0 += h;
        }
    }
    g.carry = (g.row_bands && most_splits <= g.n_vt) ? 1 : 0;
    if (g.carry) {
        plan->uniform = 0;
        plan->G = grid;
        plan->hb = g.band;
        plan->tile_rows = BLOCK_M;
        plan->n_rows = n_rows;
        plan->n_rows_dev = n_rows_dev;
    } else {
        *plan = uniform_splits(g.n_vt);
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(NUM_THREADS);
    cfg.dynamicSmemBytes = SMEM1_BYTES;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    // Starting before the kernel ahead has drained hides this kernel's set-up, which matters when the
    // whole pass takes under 200 us (one row tile).  With many row tiles an early start was measured
    // to lengthen the pass by 5-8% (8192 rows), so there the kernel keeps plain stream order.
    attr[0].val.programmaticStreamSerializationAllowed = (pdl_enabled() == 2 || (pdl_enabled() && g.n_mt == 1)) ? 1 : 0;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, confidence_tc_kernel, map_a, map_bw, map_bn, g, n_rows, H, V, part.m,
                                       part.s, part.a, status_dev, n_rows_dev, part.cap);
    count_launch();
    return e == cudaSuccess ? PSD_OK : PSD_ERR_CUDA;
}

}  // namespace psd
