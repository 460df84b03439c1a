// Work schedule of the tensor-core decode kernel: plain integer arithmetic, compiled for the device by nvcc
// and for the host by any C++ compiler (the CPU tests replay it for every cache length and check that every
// tile has exactly one owner and that the partial slots suffice).
#pragma once

#if defined(__CUDACC__)
#define MKV_HD __host__ __device__
#else
#define MKV_HD
#endif

namespace mkv {

constexpr int kSchedTile = 128;      // keys per tile

struct Item {
    int unit, tile0, nk;      // tiles [tile0, tile0 + nk) of the unit
};

// The same deterministic walk over a CTA's items in every role of the kernel.  With nt tiles per unit at
// the current cache length, global tile i is tile i % nt of unit i / nt, and CTA c of the
// E = min(grid, U * nt) working CTAs owns tiles [c * T / E, (c + 1) * T / E), T = U * nt: every
// working CTA owns at least one tile and consecutive items belong to different units.
// Order of a CTA's items: if its range ends inside a unit, that last piece comes first, then the rest in tile order.
// A unit cut by a range boundary is then worked on early by both CTAs that hold a piece of it (the one before the
// boundary starts with it, the one after it takes it first or second), so its cross-CTA merge runs while tiles
// still stream, and the item a CTA ends with is a unit all of its own, whose epilogue needs no other CTA.
struct Walk {
    int tile, tile_begin, tile_end;   // the host keeps U * tiles per unit below 2^31
    int nat_end;      // end of the part of the range that is handed out in tile order
    int lead_nk;      // tiles of the piece handed out first (0: none, or already handed out)
    int nt;           // tiles per unit
    int unit, off;    // unit and tile inside it of `tile`
    int nitems;       // items returned so far (= units seen: ring loads, partials)
    int T0;           // tiles of the items already advanced over
    int eff;          // working CTAs
    int cta;          // this CTA
    long long total;
    MKV_HD Walk(int U, int n, int grid, int cta_index)
    {
        nt = (n + kSchedTile - 1) / kSchedTile;
        total = (long long)U * nt;
        eff = (int)(total < (long long)grid ? total : (long long)grid);
        cta = cta_index;
        if (cta < eff) {
            tile = (int)(total * cta / eff);
            tile_end = (int)(total * (cta + 1) / eff);
        } else {
            tile = tile_end = 0;
        }
        tile_begin = tile;
        unit = tile / nt;         // n >= 1: a context holds at least its prompt
        off = tile - unit * nt;
        nitems = 0; T0 = 0;
        nat_end = tile_end;
        lead_nk = 0;
        if (tile_end > tile_begin) {
            const int ul = (tile_end - 1) / nt;                 // the unit the range ends in
            const int first = ul * nt;                          // its first tile
            if (tile_end != first + nt && first > tile_begin) { // the range ends inside it and starts before it
                nat_end = first;
                lead_nk = tile_end - first;
            }
        }
    }
    MKV_HD bool next(Item &x)
    {
        if (lead_nk > 0) {
            x.unit = nat_end / nt;
            x.tile0 = 0;
            x.nk = lead_nk;
            lead_nk = 0;
            return true;
        }
        if (tile >= nat_end) return false;
        x.unit = unit;
        x.tile0 = off;
        x.nk = nt - off < nat_end - tile ? nt - off : nat_end - tile;
        tile += x.nk;
        off += x.nk;
        if (off == nt) { off = 0; ++unit; }
        return true;
    }
    MKV_HD void advance(const Item &x)
    {
        T0 += x.nk;
        ++nitems;
    }
    // the CTA that owns global tile i: the largest c with c * T / E <= i
    MKV_HD int owner(long long i) const { return (int)(((i + 1) * eff - 1) / total); }
    // How many CTAs hold tiles of unit u, and this CTA's index among them.
    MKV_HD int ctas_of_unit(int u, int &my_index) const
    {
        const long long i0 = (long long)u * nt;
        const int c0 = owner(i0), c1 = owner(i0 + nt - 1);
        my_index = cta - c0;
        return c1 - c0 + 1;
    }
};

// Grid of the persistent kernel.  `splits_hint` > 0 asks for about that many CTAs per unit
// (ranges of cap_tiles / splits_hint tiles); otherwise one CTA per SM.
inline int sched_grid(int U, int cap, int splits_hint, int n_sm)
{
    const long long ntiles = (cap + kSchedTile - 1) / kSchedTile, total = (long long)U * ntiles;
    long long grid = n_sm;
    if (splits_hint > 0) {
        const long long chunk = (ntiles + splits_hint - 1) / splits_hint;
        grid = (total + chunk - 1) / chunk;
        if (grid > n_sm) grid = n_sm;
    }
    if (grid > total) grid = total;
    return (int)(grid < 1 ? 1 : grid);
}

// Upper bound, over every cache length up to cap, of the CTAs that hold tiles of one unit
// (= partial slots a unit needs).
inline int sched_partials_per_unit(int U, int cap, int grid)
{
    const int ntiles = (cap + kSchedTile - 1) / kSchedTile;
    int worst = 1;
    for (int nt = 1; nt <= ntiles; ++nt) {
        const long long total = (long long)U * nt;
        const long long eff = total < grid ? total : grid;
        const long long len = total / eff;                     // shortest range of a CTA
        long long c = (nt + len - 1) / len + 1;
        if (c > nt) c = nt;
        if (c > worst) worst = (int)c;
    }
    return worst;
}

}  // namespace mkv
