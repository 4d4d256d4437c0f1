// Fused LM-head + confidence kernel for sm_100a, CTA-pair version (Sec. 3.1: x^ = argmax_v p(v),
// c = max_v p(v)).
//
// Two CTAs on neighbouring SMs (a cluster of 2) work on one tile of 256 rows x up to 256 vocabulary
// entries with tcgen05.mma.cta_group::2 (M = 256): each CTA stages its own 128 rows of `hidden` and
// its own HALF of the W tile, and the tensor cores of both SMs read both halves.  Per 128 x 256 block
// of logits that is 32 KB per K-slice through L2 and shared memory instead of the single-CTA
// kernel's 48 KB.  Each CTA keeps the accumulator of its 128 rows in its own TMEM and runs the same
// epilogue as the single-CTA kernel (thread = row, online max / sum-exp / argmax, partial triples
// carried per row tile of a band and written at the band's end, see SplitPlan).  Logits never leave
// the SM.
//
// Measured on B200 (V = 126464, H = 4096) this version moves a third less data from L2 to the SMs
// (66 GB against 99 GB per 8192-row pass) and runs within 2% of the single-CTA kernel from 512 to 8192
// rows once the board sits at its power cap.  Where it wins is 129..256 rows: one pair covers both row
// tiles, so every W tile is fetched once and by one pair, and that range is where the default uses it;
// elsewhere it is selected with psd_set_confidence_impl(3).  It is held to the same parity tests.
//
// Roles per CTA: warp 0 = TMA producer (own operands), warp 1 = TMEM allocation, and in the leader
// CTA (cluster rank 0) the MMA issuer for the pair, warps 2-5 = epilogue.  Barriers:
//   full[s]      leader only; both CTAs' TMA copies complete their bytes on it
//   empty[s]     one in each CTA; the leader's tcgen05.commit arrives on both
//   acc_full[a]  one in each CTA; the leader's tcgen05.commit arrives on both
//   acc_empty[a] leader only; the 8 epilogue warps of the pair arrive on it
// No TMA load is multicast.  Every wait is bounded as in the single-CTA kernel; both CTAs meet at a
// cluster barrier before they free TMEM and exit, so neither touches the other's shared memory after
// that CTA has gone.
#include <algorithm>
#include "tc_common.cuh"

namespace psd {
namespace {

#ifndef PSD_STAGES2
#define PSD_STAGES2 6
#endif
constexpr int STAGES2 = PSD_STAGES2;               // depth of the shared-memory ring (32 KB per stage)
constexpr int HALF_N = BLOCK_N / 2;                  // widest half tile of W held by one CTA
constexpr int B2_BYTES = HALF_N * BLOCK_K * 2;       // 16 KB
constexpr int STAGE2_BYTES = A_BYTES + B2_BYTES;     // 32 KB
constexpr long long PAIR_DRAIN_CYCLES = 100000000ll;  // about 50 ms: how long an aborting leader watches one slice
constexpr int BARRIER2_BYTES = 256;
constexpr int CARRY2_BYTES = kCarryEntries * BLOCK_M * 12;   // carried triples of a CTA (24 KB)
constexpr int SMEM2_BYTES = STAGES2 * STAGE2_BYTES + 1024 /* alignment slack */ + BARRIER2_BYTES + CARRY2_BYTES;
static_assert(SMEM2_BYTES <= 227 * 1024, "shared memory of the CTA-pair kernel");

__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// Address, in the cluster's shared window, of the same shared-memory location in CTA `rank`.
__device__ __forceinline__ uint32_t map_to_cta(uint32_t smem_addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait_cluster(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait on a barrier that threads of the other CTA arrive on.
__device__ __forceinline__ bool mbar_wait_cluster(uint64_t* bar, uint32_t parity, const WaitCtx& w) {
    if (mbar_try_wait_cluster(bar, parity)) return true;
    const long long t0 = clock64();
    for (;;) {
        for (int i = 0; i < 256; ++i)
            if (mbar_try_wait_cluster(bar, parity)) return true;
        if (*w.abort_flag) return false;
        if (clock64() - t0 > w.limit) {
            raise_abort(w);
            return false;
        }
    }
}

// TMA tile load issued by one CTA of a pair into its own shared memory; the bytes are counted on
// `bar_cluster_addr`, which may be a barrier of the other CTA of the pair.  Not a multicast.
__device__ __forceinline__ void tma_load_2d_pair(void* smem_dst, const CUtensorMap* map, uint32_t bar_cluster_addr,
                                                 int x, int y, uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
        " [%0], [%1, {%3, %4}], [%2], %5;"
        ::"r"(smem_u32(smem_dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar_cluster_addr), "r"(x), "r"(y),
        "l"(policy)
        : "memory");
}

// Instruction descriptor, kind::f16, for the pair: D = fp32, A = B = bf16, K-major, M = 256, N = n.
__device__ __forceinline__ uint32_t umma_idesc_pair(int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);
}

__device__ __forceinline__ void umma_f16_pair(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc,
                                              uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
        : "memory");
}

// Arrives on the barrier at this shared-memory offset in BOTH CTAs of the pair once every MMA issued
// so far by this thread has completed.
__device__ __forceinline__ void umma_commit_pair(uint64_t* bar) {
    const uint16_t both = 3;
    asm volatile(
        "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
        ::"r"(smem_u32(bar)), "h"(both) : "memory");
}

__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(NUM_THREADS, 1)
confidence_tc2_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b_wide,
                      const __grid_constant__ CUtensorMap map_b_narrow, TileGeometry geo, int n_rows, int H, int V,
                      float* __restrict__ pm, float* __restrict__ ps, int32_t* __restrict__ pa,
                      int32_t* status_dev, const int32_t* __restrict__ n_rows_dev, size_t part_cap) {
    extern __shared__ unsigned char smem_raw[];
    // 1024-byte alignment for the 128-byte swizzle; the dynamic shared memory of both CTAs of a cluster
    // starts at the same offset, so the aligned layouts coincide, as cta_group::2 addressing requires.
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                                           ~static_cast<uintptr_t>(1023));
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + STAGES2 * STAGE2_BYTES);
    uint64_t* full_bar = bars;                     // [STAGES2] used in the leader
    uint64_t* empty_bar = bars + STAGES2;          // [STAGES2]
    uint64_t* acc_full_bar = bars + 2 * STAGES2;   // [2]
    uint64_t* acc_empty_bar = acc_full_bar + 2;    // [2] used in the leader
    uint64_t* drain_bar = acc_empty_bar + 2;       // [1] used only when aborting
    uint64_t* never_bar = drain_bar + 1;           // [1] nothing ever arrives on it (self-test of the give-up path)
    uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(never_bar + 1);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);
#ifdef PSD_DEBUG
    volatile int* ring_tag = abort_flag + 1;   // [stages] the K-slice number the loader put in each stage
#endif
    // carried triples: [kCarryEntries][BLOCK_M] max, then sum-exp, then argmax
    float* carry_m = reinterpret_cast<float*>(smem + STAGES2 * STAGE2_BYTES + BARRIER2_BYTES);
    float* carry_s = carry_m + kCarryEntries * BLOCK_M;
    int32_t* carry_a = reinterpret_cast<int32_t*>(carry_s + kCarryEntries * BLOCK_M);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const bool leader = rank == 0;
    const int pair_id = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
    const int k_blocks = H / BLOCK_K;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES2; ++s) {
            mbar_init(&full_bar[s], 1);     // the leader's producer arrives (with the byte count of both CTAs)
            mbar_init(&empty_bar[s], 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(&acc_full_bar[a], 1);
            mbar_init(&acc_empty_bar[a], 8);   // one arrival per epilogue warp of the pair
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
        // TMEM for a CTA pair is allocated by one warp of each of the two CTAs.
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(tmem_holder)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncwarp();
    cluster_sync_all();   // barriers of both CTAs are initialised before either CTA signals the other
    tc_fence_after();
    const uint32_t tmem_base = *tmem_holder;

    asm volatile("griddepcontrol.wait;" ::: "memory");

    // rows known only on the device (see the single-CTA kernel): the tile list shrinks accordingly
    int n_rows_act = n_rows;
    if (n_rows_dev) {
        n_rows_act = min(max(*n_rows_dev, 0), n_rows);
        geo.n_mt = (n_rows_act + 2 * BLOCK_M - 1) / (2 * BLOCK_M);
    }
    const int n_mt = geo.n_mt;
    // a wait that runs out raises the abort flag of BOTH CTAs of the pair, so they give up together
    const WaitCtx wc = {abort_flag, status_dev, geo.wait_limit,
                        map_to_cta(smem_u32(const_cast<int*>(abort_flag)), rank ^ 1u)};

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (each CTA)
        if (lane == 0) {
            // both operands are re-read from L2 many times within a band: mark both to stay (as in the
            // single-CTA kernel with several row tiles)
            const uint64_t pol_w = l2_policy_evict_last();
            const uint64_t pol_h = l2_policy_evict_last();
            const uint32_t full0 = map_to_cta(smem_u32(&full_bar[0]), 0);   // the leader's full[0]
            int q = 0;
            bool ok = true;
            TileCursor cur;
            cur.begin(geo, pair_id, n_pairs, n_mt);
            for (int ev; ok && (ev = cur.next(geo)) != TileCursor::DONE;) {
                if (ev != TileCursor::TILE) continue;
                const int m_tile = cur.m_tile, v_tile = cur.v_tile, v0 = cur.v0, ncols = cur.ncols;
                const bool wide = v_tile < geo.rem || geo.rem == 0;
                const CUtensorMap* mb = wide ? &map_b_wide : &map_b_narrow;
                const int half = ncols >> 1;
                const uint32_t bytes_pair = 2u * (A_BYTES + (uint32_t)half * BLOCK_K * 2);
                const int row0 = m_tile * 256 + (int)rank * BLOCK_M;
                const int col0 = v0 + (int)rank * half;
                for (int kb = 0; kb < k_blocks; ++kb, ++q) {
                    const int s = q % STAGES2;
                    if (!mbar_wait(&empty_bar[s], ((q / STAGES2) & 1) ^ 1, wc)) { ok = false; break; }
                    // the partner may have given up while this stage was free: issue nothing more then
                    if (*abort_flag) { ok = false; break; }
                    unsigned char* sa = smem + s * STAGE2_BYTES;
#ifdef PSD_DEBUG
                    if (leader) ring_tag[s] = q;
#endif
                    if (leader) mbar_arrive_expect_tx(&full_bar[s], bytes_pair);
                    const uint32_t fb = full0 + (uint32_t)s * 8;
                    tma_load_2d_pair(sa, &map_a, fb, kb * BLOCK_K, row0, pol_h);
                    tma_load_2d_pair(sa + A_BYTES, mb, fb, kb * BLOCK_K, col0, pol_w);
                    // self-test of the give-up path (leading CTA only): a wait that nothing will ever satisfy
                    if (geo.stall_test && leader && q == 0 && !mbar_wait(never_bar, 0, wc)) { ok = false; ++q; break; }
                }
            }
            if (!ok) {
                // Aborting: no copy may still be in flight when the CTA exits.  The leader can watch its
                // full barriers (bounded; a slice whose other half the partner never sent runs that wait
                // out); the other CTA's copies report to the leader's barriers, which it cannot poll, so
                // it lets a fixed interval pass that is far longer than any copy takes.  Both CTAs stay
                // resident until the cluster barrier at the end, so a late byte count still finds its barrier.
                if (leader) {
                    const int first = q > STAGES2 ? q - STAGES2 : 0;
                    for (int i = first; i < q; ++i) {
                        const long long t0 = clock64();
                        while (!mbar_try_wait(&full_bar[i % STAGES2], (i / STAGES2) & 1) &&
                               clock64() - t0 < PAIR_DRAIN_CYCLES) {}
                    }
                } else {
                    const long long t0 = clock64();
                    while (clock64() - t0 < 2000000ll) {}
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (leader only)
        if (leader && lane == 0) {
            int q = 0, it = 0;
            bool ok = true;
            TileCursor cur;
            cur.begin(geo, pair_id, n_pairs, n_mt);
            for (int ev; ok && (ev = cur.next(geo)) != TileCursor::DONE;) {
                if (ev != TileCursor::TILE) continue;
                const int acc = it & 1;
                if (!mbar_wait_cluster(&acc_empty_bar[acc], ((it >> 1) & 1) ^ 1, wc)) { ok = false; break; }
                tc_fence_after();
                const uint32_t idesc = umma_idesc_pair(cur.ncols);
                const uint32_t tmem_d = tmem_base + (uint32_t)(acc * BLOCK_N);
                for (int kb = 0; kb < k_blocks; ++kb, ++q) {
                    const int s = q % STAGES2;
                    if (!mbar_wait(&full_bar[s], (q / STAGES2) & 1, wc)) { ok = false; break; }
                    tc_fence_after();
#ifdef PSD_DEBUG
                    PSD_DEBUG_OK(ring_tag[s] == q, status_dev);   // the stage holds the slice this MMA expects
#endif
                    const uint32_t a_addr = smem_u32(smem + s * STAGE2_BYTES);
                    const uint64_t da = umma_smem_desc(a_addr);
                    const uint64_t db = umma_smem_desc(a_addr + A_BYTES);
#pragma unroll
                    for (int k = 0; k < BLOCK_K / UMMA_K; ++k)
                        umma_f16_pair(tmem_d, da + (uint64_t)(k * 2), db + (uint64_t)(k * 2), idesc, (kb | k) != 0);
                    umma_commit_pair(&empty_bar[s]);
                }
                if (ok) umma_commit_pair(&acc_full_bar[acc]);
                ++it;
            }
            if (!ok) {
                umma_commit_pair(drain_bar);   // nothing may still be writing TMEM when it is freed
                const long long t0 = clock64();
                while (!mbar_try_wait(drain_bar, 0) && clock64() - t0 < WAIT_LIMIT_CYCLES) {}
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2..5, each CTA)
        const int quarter = warp & 3;
        const int row_in_tile = quarter * 32 + lane;
        const uint32_t acc_empty0 = map_to_cta(smem_u32(&acc_empty_bar[0]), 0);   // the leader's acc_empty[0]
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
        cur.begin(geo, pair_id, n_pairs, n_mt);
        for (int ev; ok && (ev = cur.next(geo)) != TileCursor::DONE;) {
            if (ev == TileCursor::BAND_END) {
                // The band is over for this pair: each CTA writes the triples it carried for its half of
                // every row tile of the pair's residue class, to the pair's slot of those rows.
                const int entries = cur.end_h / cur.end_gcd;
                const int slot = pair_id / cur.end_gcd, base = pair_id % cur.end_gcd;
                for (int e = 0; e < entries; ++e) {
                    const int row = (cur.end_m0 + base + e * cur.end_gcd) * 256 + (int)rank * BLOCK_M + row_in_tile;
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
            // a pair meets the tiles of one row tile in ascending vocabulary order: a carried triple keeps the
            // lowest index among equal maxima
            const int entry = geo.carry ? ((m_tile - cur.m0) / cur.gcd) * BLOCK_M + row_in_tile : 0;
            if (!PSD_DEBUG_OK(m_tile >= 0 && m_tile < n_mt && v0 >= 0 && v0 < V && ncols > 0 && ncols <= BLOCK_N &&
                                  entry >= 0 && entry < kCarryEntries * BLOCK_M, status_dev)) { ok = false; break; }
            float run_m = -INFINITY, run_s = 0.f;
            int run_a = 0;
            if (geo.carry) { run_m = carry_m[entry]; run_s = carry_s[entry]; run_a = carry_a[entry]; }
            const bool ragged = v0 + ncols > V;
            for (int c = 0; c < ncols; c += 32) {
                float x[32];
                tmem_ld_32x32(taddr + c, x);     // tile widths are multiples of 32 here
                if (ragged) {
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        if (v0 + c + j >= V) x[j] = -INFINITY;
                }
                fold_chunk(x, v0 + c, run_m, run_s, run_a);
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(acc_empty0 + (uint32_t)acc * 8);
            if (geo.carry) {
                carry_m[entry] = run_m; carry_s[entry] = run_s; carry_a[entry] = run_a;
            } else {
                const int row = m_tile * 256 + (int)rank * BLOCK_M + row_in_tile;
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
    __syncwarp();
    cluster_sync_all();   // both CTAs are done with each other's shared memory and with TMEM
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

}  // namespace

int launch_confidence_tc2(const void* hidden, const void* w, int n_rows, int H, int V, Partials part,
                          int32_t* status_dev, const int32_t* n_rows_dev, cudaStream_t st, SplitPlan* plan) {
    static std::atomic<unsigned long long> smem_set{0};
    if (!ensure_dynamic_smem(confidence_tc2_kernel, SMEM2_BYTES, smem_set)) return PSD_ERR_CUDA;
    const int pairs_max = sm_count() / 2;
    TileGeometry g = choose_geometry(n_rows, V, pairs_max, max_splits(V), 2 * BLOCK_M, 32);
    choose_order(g, n_rows, H, V, 2 * BLOCK_M, band_bytes(), tile_order());
    if (g.n_mt == 1) { g.row_bands = 1; g.band = 1; }   // one row tile: ascending vocabulary order either way
    const int wide_half = (g.rem ? g.base_units + 1 : g.base_units) * 16;      // half of unit 32
    const int narrow_half = g.base_units > 0 ? g.base_units * 16 : wide_half;
    CUtensorMap map_a, map_bw, map_bn;
    if (!make_map(&map_a, hidden, n_rows, H, BLOCK_M) || !make_map(&map_bw, w, V, H, wide_half) ||
        !make_map(&map_bn, w, V, H, narrow_half))
        return PSD_ERR_CUDA;
    const int n_tiles = g.n_mt * g.n_vt;
    const int pairs = n_tiles < pairs_max ? n_tiles : pairs_max;
    // carried partials under the same conditions as in the single-CTA launcher
    int most_splits = pairs;
    if (!n_rows_dev) {
        most_splits = 0;
        for (int m0 = 0; m0 < g.n_mt;) {
            const int h = band_height(pairs, g.band, g.n_mt - m0);
            most_splits = std::max(most_splits, pairs / gcd_int(pairs, h));
            m0 += h;
        }
    }
    g.carry = (g.row_bands && most_splits <= g.n_vt) ? 1 : 0;
    if (g.carry) {
        plan->uniform = 0;
        plan->G = pairs;
        plan->hb = g.band;
        plan->tile_rows = 2 * BLOCK_M;
        plan->n_rows = n_rows;
        plan->n_rows_dev = n_rows_dev;
    } else {
        *plan = uniform_splits(g.n_vt);
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * pairs);
    cfg.blockDim = dim3(NUM_THREADS);
    cfg.dynamicSmemBytes = SMEM2_BYTES;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    // early start only for one row tile, as in the single-CTA launcher
    attr[0].val.programmaticStreamSerializationAllowed = (pdl_enabled() == 2 || (pdl_enabled() && g.n_mt == 1)) ? 1 : 0;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, confidence_tc2_kernel, map_a, map_bw, map_bn, g, n_rows, H, V, part.m,
                                       part.s, part.a, status_dev, n_rows_dev, part.cap);
    count_launch();
    return e == cudaSuccess ? PSD_OK : PSD_ERR_CUDA;
}

}  // namespace psd
