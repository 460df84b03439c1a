// Replays the tensor-core decode kernel's work schedule on the host, for every number of tiles per unit up to the
// capacity, and checks what the kernel relies on:
//   - every tile of every unit is owned by exactly one CTA, and a CTA's tiles are one contiguous range (handed out
//     with the piece of a unit at the end of the range first, the rest in tile order);
//   - a CTA's consecutive items belong to different units (one ring load and one partial per item);
//   - ctas_of_unit() agrees with the CTAs that really hold tiles of the unit (the ticket count of the unit's
//     epilogue), and their indices are 0 .. ncta-1 in CTA order;
//   - an index is always below the partial slots the host allocated (sched_partials_per_unit);
//   - key rows stay below the capacity rounded up to a tile (the tensor maps clip at the capacity).
// usage: schedule_replay U cap splits_hint n_sm    -> prints "ok <grid> <splits> <checked tiles>" or a diagnostic
#include <cstdio>
#include <cstdlib>
#include <vector>

#include "mkv_schedule.h"

using namespace mkv;

int main(int argc, char **argv)
{
    if (argc != 5) { fprintf(stderr, "usage: %s U cap splits_hint n_sm\n", argv[0]); return 2; }
    const int U = atoi(argv[1]), cap = atoi(argv[2]), hint = atoi(argv[3]), n_sm = atoi(argv[4]);
    const int grid = sched_grid(U, cap, hint, n_sm);
    const int splits = sched_partials_per_unit(U, cap, grid);
    const int ntiles = (cap + kSchedTile - 1) / kSchedTile;
    long long checked = 0;
    for (int nt = 1; nt <= ntiles; ++nt) {
        // the schedule depends on n only through the tiles per unit: the shortest and the longest n of this count
        const int n_lo = (nt - 1) * kSchedTile + 1, n_hi = nt * kSchedTile < cap ? nt * kSchedTile : cap;
        for (int n : {n_lo, n_hi}) {
            std::vector<int> owner((size_t)U * nt, -1);
            std::vector<int> holders(U, 0);              // CTAs that hold tiles of the unit, counted from the walk
            std::vector<int> next_index(U, 0);
            for (int cta = 0; cta < grid; ++cta) {
                Walk w(U, n, grid, cta);
                Item x;
                int prev_unit = -1, seen = 0;
                long long got_tiles = 0, expect_tile = w.tile_begin;
                const bool lead = w.lead_nk > 0;
                while (w.next(x)) {
                    if (x.unit < 0 || x.unit >= U || x.nk < 1 || x.tile0 < 0 || x.tile0 + x.nk > nt) {
                        printf("bad item: n=%d cta=%d unit=%d tile0=%d nk=%d\n", n, cta, x.unit, x.tile0, x.nk);
                        return 1;
                    }
                    if (x.unit == prev_unit) { printf("n=%d cta=%d: two items of unit %d in a row\n", n, cta, x.unit); return 1; }
                    const long long g0 = (long long)x.unit * nt + x.tile0;
                    if (g0 < w.tile_begin || g0 + x.nk > w.tile_end) { printf("n=%d cta=%d: item outside the CTA's range\n", n, cta); return 1; }
                    if (lead && seen == 0) {
                        // the piece at the end of the range: a proper part of its unit, starting at the unit's first tile
                        if (x.tile0 != 0 || x.nk >= nt || g0 + x.nk != w.tile_end) { printf("n=%d cta=%d: bad leading piece\n", n, cta); return 1; }
                    } else {
                        if (g0 != expect_tile) { printf("n=%d cta=%d: range not in tile order\n", n, cta); return 1; }
                        expect_tile += x.nk;
                    }
                    got_tiles += x.nk;
                    if ((x.tile0 + x.nk) * kSchedTile > ntiles * kSchedTile) { printf("n=%d cta=%d: key row beyond the capacity\n", n, cta); return 1; }
                    for (int j = 0; j < x.nk; ++j) {
                        int &o = owner[(size_t)x.unit * nt + x.tile0 + j];
                        if (o != -1) { printf("n=%d: tile %d of unit %d owned by CTAs %d and %d\n", n, x.tile0 + j, x.unit, o, cta); return 1; }
                        o = cta;
                        if (w.owner((long long)x.unit * nt + x.tile0 + j) != cta) { printf("n=%d: owner() disagrees with the walk\n", n); return 1; }
                    }
                    int my_index = -1;
                    const int ncta = w.ctas_of_unit(x.unit, my_index);
                    if (my_index != next_index[x.unit]) { printf("n=%d cta=%d unit=%d: index %d, expected %d\n", n, cta, x.unit, my_index, next_index[x.unit]); return 1; }
                    if (my_index < 0 || my_index >= ncta || my_index >= splits) {
                        printf("n=%d cta=%d unit=%d: index %d of %d CTAs with %d partial slots\n", n, cta, x.unit, my_index, ncta, splits);
                        return 1;
                    }
                    ++next_index[x.unit];
                    ++holders[x.unit];
                    prev_unit = x.unit;
                    w.advance(x);
                    ++seen;
                }
                if (got_tiles != w.tile_end - w.tile_begin) { printf("n=%d cta=%d: walk stopped early\n", n, cta); return 1; }
                if (w.nitems != seen || w.T0 != w.tile_end - w.tile_begin) { printf("n=%d cta=%d: counters off\n", n, cta); return 1; }
            }
            for (size_t i = 0; i < owner.size(); ++i)
                if (owner[i] < 0) { printf("n=%d: tile %zu has no owner\n", n, i); return 1; }
            Walk any(U, n, grid, 0);
            for (int u = 0; u < U; ++u) {
                int idx;
                if (any.ctas_of_unit(u, idx) != holders[u]) { printf("n=%d unit=%d: ctas_of_unit %d, holders %d\n", n, u, any.ctas_of_unit(u, idx), holders[u]); return 1; }
            }
            checked += (long long)U * nt;
        }
    }
    printf("ok %d %d %lld\n", grid, splits, checked);
    return 0;
}
