// Host-side check of the tile walk of the tensor-core kernels, run on the CPU by
// tests/test_host_tile_plan.py: the very functions the kernels use (choose_geometry, choose_order,
// TileCursor, band_height, carried_splits) are compiled for the host and every CTA's walk is replayed.
// Checked for many shapes: every (row tile, vocabulary tile) is visited exactly once; a CTA meets the
// tiles of one row tile in ascending vocabulary order and carries at most kCarryEntries row tiles per
// band; the slots a band's CTAs write for a row tile are exactly 0 .. carried_splits - 1, once each;
// the vocabulary tiles cover [0, V) without gap or overlap.
#include <cstdio>
#include <cstdlib>
#include <map>
#include <set>
#include <vector>
#include "tc_common.cuh"

namespace psd {
// the two settings the geometry reads from the library's knobs
long long wait_limit_cycles() { return WAIT_LIMIT_CYCLES; }
int selftest_stall() { return 0; }
}  // namespace psd

using namespace psd;

static int failures = 0;
#define CHECK(cond, ...)                                                     \
    do {                                                                     \
        if (!(cond)) {                                                       \
            if (failures < 20) { std::printf("FAIL %s: ", #cond); std::printf(__VA_ARGS__); std::printf("\n"); } \
            ++failures;                                                      \
        }                                                                    \
    } while (0)

static void check_case(int n_rows, int H, int V, int workers, int tile_rows, int unit, long long budget, int force,
                       int carry) {
    TileGeometry g = choose_geometry(n_rows, V, workers, max_splits(V), tile_rows, unit);
    choose_order(g, n_rows, H, V, tile_rows, budget, force);
    if (g.n_mt == 1) { g.row_bands = 1; g.band = 1; }
    g.carry = (carry && g.row_bands) ? 1 : 0;
    const int n_tiles = g.n_mt * g.n_vt;
    const int G = n_tiles < workers ? n_tiles : workers;
    // the vocabulary tiles partition [0, V) (the last one may reach past V by less than its width)
    int next_col = 0;
    for (int v = 0; v < g.n_vt; ++v) {
        int v0, nc;
        tile_columns(g, v, v0, nc);
        CHECK(v0 == next_col && nc > 0 && nc <= BLOCK_N && nc % unit == 0, "V=%d tile %d: v0 %d ncols %d", V, v, v0, nc);
        next_col = v0 + nc;
    }
    CHECK(next_col >= V && next_col - V < 2 * unit * 16, "V=%d covered up to %d", V, next_col);

    std::vector<int> seen((size_t)n_tiles, 0);
    std::map<int, std::vector<int>> slots;   // row tile -> slots written at band ends
    for (int c = 0; c < G; ++c) {
        TileCursor cur;
        cur.begin(g, c, G, g.n_mt);
        std::map<int, int> last_v;           // row tile -> last vocabulary tile met in this band
        std::set<int> entries;
        for (int ev; (ev = cur.next(g)) != TileCursor::DONE;) {
            if (ev == TileCursor::BAND_END) {
                CHECK(g.carry, "band end without carried partials");
                const int n_e = cur.end_h / cur.end_gcd;
                CHECK(n_e <= kCarryEntries && cur.end_h % cur.end_gcd == 0 && G % cur.end_gcd == 0, "entries %d", n_e);
                for (int e = 0; e < n_e; ++e) {
                    const int m = cur.end_m0 + c % cur.end_gcd + e * cur.end_gcd;
                    CHECK(m < cur.end_m0 + cur.end_h && m < g.n_mt, "flush of row tile %d", m);
                    slots[m].push_back(c / cur.end_gcd);
                }
                for (int e : entries) CHECK(e < n_e, "entry %d of %d", e, n_e);
                last_v.clear();
                entries.clear();
                continue;
            }
            CHECK(cur.m_tile >= 0 && cur.m_tile < g.n_mt && cur.v_tile >= 0 && cur.v_tile < g.n_vt, "tile (%d, %d)",
                  cur.m_tile, cur.v_tile);
            if (cur.m_tile < 0 || cur.m_tile >= g.n_mt || cur.v_tile < 0 || cur.v_tile >= g.n_vt) continue;
            ++seen[(size_t)cur.m_tile * g.n_vt + cur.v_tile];
            if (g.carry) {
                CHECK((cur.m_tile - cur.m0) % cur.gcd == c % cur.gcd, "row tile %d outside the CTA's class", cur.m_tile);
                entries.insert((cur.m_tile - cur.m0) / cur.gcd);
                auto it = last_v.find(cur.m_tile);
                CHECK(it == last_v.end() || it->second < cur.v_tile, "vocabulary order of row tile %d", cur.m_tile);
                last_v[cur.m_tile] = cur.v_tile;
            }
        }
    }
    for (int t = 0; t < n_tiles; ++t) CHECK(seen[t] == 1, "rows %d V %d: tile %d visited %d times", n_rows, V, t, seen[t]);
    if (g.carry) {
        for (int m = 0; m < g.n_mt; ++m) {
            const int ns = carried_splits(G, g.band, g.n_mt, m);
            std::vector<int>& s = slots[m];
            std::set<int> u(s.begin(), s.end());
            CHECK((int)s.size() == ns && (int)u.size() == ns && (u.empty() || (*u.begin() == 0 && *u.rbegin() == ns - 1)),
                  "rows %d V %d G %d band %d: row tile %d has %d slots, expected %d", n_rows, V, G, g.band, m,
                  (int)s.size(), ns);
        }
    }
}

int main() {
    const int Vs[] = {1, 17, 300, 1024, 3001, 30001, 126464, 152064};
    const int Rs[] = {1, 127, 128, 129, 256, 300, 384, 512, 1024, 1500, 1536, 2048, 4096, 4480, 8192, 9100, 70000};
    const long long budgets[] = {0, 70000, 300000, 36ll << 20};
    int cases = 0;
    for (int V : Vs)
        for (int R : Rs) {
            if ((long long)R * V > 3000000000ll) continue;                    // keeps the replay short
            for (long long budget : budgets)
                for (int force = 0; force <= 2; ++force)
                    for (int carry = 0; carry <= 1; ++carry) {
                        check_case(R, 4096, V, 148, BLOCK_M, 16, budget, force, carry);        // single-CTA kernel
                        check_case(R, 4096, V, 74, 2 * BLOCK_M, 32, budget, force, carry);     // CTA pairs
                        check_case(R, 128, V, 132, BLOCK_M, 16, budget, force, carry);         // another SM count
                        cases += 3;
                    }
        }
    // band heights: never more than kCarryEntries row tiles per CTA, always progress
    for (int G = 1; G <= 160; ++G)
        for (int hb = 1; hb <= 600; hb += 7)
            for (int rem = 1; rem <= 600; rem += 11) {
                const int h = band_height(G, hb, rem);
                CHECK(h >= 1 && h <= hb && h <= rem && h / gcd_int(G, h) <= kCarryEntries, "band_height(%d,%d,%d)=%d", G, hb, rem, h);
            }
    std::printf("%s: %d cases, %d failures\n", failures ? "FAILED" : "ok", cases, failures);
    return failures ? 1 : 0;
}
