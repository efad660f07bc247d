// Mapping of chunks to work items for the general worker and server kernels.
// Part of libapms.so: included by apms.cu, which is the only translation unit.
#pragma once

namespace {

// ------------------------------------------------------------------------------------------
// Mapping of chunks to work items.  An item is one tile of one chunk (for one worker on the
// worker side).  Chunks up to kTileMax elements are one tile; longer chunks (the paper's own
// layout is chunk = d/n) are cut into tiles of kTileSplit elements whose binary64 partial sums
// of squares go to a scratch array and are added up, in tile order, by k_finalize_scales.
// A team of WPC warps works on an item: the whole CTA (WPC = 8) or, for short chunks, one warp
// (WPC = 1, eight items per CTA and no CTA-wide barrier).

constexpr int64_t kTileMax = 65536;
constexpr int64_t kTileSplit = 32768;
// A tile is given to a single warp (eight tiles per CTA, no CTA-wide barrier) whenever that
// still leaves at least kWarpTeamMinCtasPerSm CTAs per SM; small problems use one CTA per tile.
constexpr int kWarpTeamMinCtasPerSm = 6;

struct Tiling {
    int64_t d, chunk, tile;   // tile == chunk when P == 1
    int P;                    // tiles per chunk
    int64_t Pp;               // row stride of the partial-sum arrays (>= C * P)
    int l1 = 0;               // scale = mean |z| instead of ||z||_2 / sqrt(L)
};

struct Item { int64_t c; int p; int64_t base; int L; int Lc; };

__device__ __forceinline__ Item decode_item(const Tiling& t, int64_t chunk_tile)
{
    Item it;
    it.p = (t.P == 1) ? 0 : (int)(chunk_tile % t.P);
    it.c = (t.P == 1) ? chunk_tile : chunk_tile / t.P;
    const int64_t cbeg = it.c * t.chunk;
    const int64_t cend = (t.d - cbeg < t.chunk) ? t.d : cbeg + t.chunk;
    it.base = cbeg + (int64_t)it.p * t.tile;
    const int64_t left = cend - it.base;
    it.L = (int)(left < t.tile ? (left > 0 ? left : 0) : t.tile);
    it.Lc = (int)(cend - cbeg);
    return it;
}

template <int WPC>
__device__ __forceinline__ double team_sum(double a, double* smem)
{
    if (WPC == 1) return warp_sum(a);      // valid in lane 0
    return block_sum(a, smem);             // valid in thread 0
}

}  // namespace
