// Tile order and per-pair tile ranges of the CTA-pair GEMM kernels (host and device).
#pragma once

namespace nm {

// Order of the tiles of the pair kernel.  Token tiles are cut into bands of `band` tiles; inside a band the
// tiles run output-tile-major.  With band = n_tok_tiles this is the plain output-tile-major order (one
// long run per output tile: weights and metadata change rarely).  A band of about one pair's share
// makes neighbouring pairs work on the SAME token tiles of different output tiles at the same time, so
// that X is fetched from DRAM once and found in L2 by the others.
struct TileCoord { int o, t; };
__host__ __device__ inline TileCoord tile_coord(int tile, int n_tok_tiles, int n_out_tiles, int band) {
    const int per_band = band * n_out_tiles;
    const int b = tile / per_band, r = tile - b * per_band;
    const int rest = n_tok_tiles - b * band, tb = band < rest ? band : rest;  // the last band may be short
    const int o = r / tb;
    return TileCoord{o, b * band + (r - o * tb)};
}

// Tile ranges of the CTA pairs, computed on the host: start[p] .. start[p + 1] is pair p's range.  A pair
// whose range crosses into a new output tile stalls there (weights and metadata are replaced once
// the MMAs of the old one have drained), so such a range is made shorter by that cost.
constexpr int kMaxPairs = 128;
struct PairSchedule {
    int start[kMaxPairs + 1];
};

// Tile plan of the pair kernel: the band size of the tile order (returned) and start[0..pairs], the contiguous
// range of every pair.  Resident weights: one long run per output tile (band = all token tiles).  Streamed
// weights: bands of about one pair's share, unless `band_request` > 0 asks for another size.  The ranges
// have about equal cost, a tile costing 1 and an output-tile change inside a range `crossing` tiles.
inline int plan_pair_tiles(int n_tok_tiles, int n_out_tiles, int pairs, bool resident, int band_request, int* start) {
    const int n_tiles = n_tok_tiles * n_out_tiles;
    int band = n_tok_tiles;
    if (!resident) {
        const int b = band_request > 0 ? band_request : (n_tiles + pairs / 2) / pairs;
        band = b < 1 ? 1 : (b > n_tok_tiles ? n_tok_tiles : b);
    }
    const double crossing = resident ? 1.0 : 0.2;
    auto out_of = [&](int t) { return tile_coord(t, n_tok_tiles, n_out_tiles, band).o; };
    auto cost = [&](int t) { return 1.0 + ((t > 0 && out_of(t) != out_of(t - 1)) ? crossing : 0.0); };
    double total = 0.0;
    for (int t = 0; t < n_tiles; ++t) total += cost(t);
    int t = 0;
    double before = 0.0;  // cost of the tiles before t
    for (int q = 0; q < pairs; ++q) {
        const double threshold = q * total / pairs;
        while (t < n_tiles - (pairs - q) && before + 0.5 * cost(t) < threshold) before += cost(t++);
        if (q > 0 && t <= start[q - 1]) before += cost(t++);  // every pair gets at least one tile
        start[q] = t;
    }
    start[pairs] = n_tiles;
    return band;
}

}  // namespace nm
