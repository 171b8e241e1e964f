// Tile lookup for the kernels that work on segments (per-layer scale) or on buckets larger
// than one CTA tile.
#pragma once

#include "mqg_common.cuh"
#include "mqg_internal.h"

namespace mqg {

struct SegQuantArgs {
    const void* grad;
    uint32_t* codes;
    float* scales;          // scale of segment j at scales[j]
    uint64_t elem_offset;
    DrawKey key;
};

// The encode pass of the segment quantizers: one CTA per tile, scale of the tile's segment read
// from a.scales (already final, or the raw maximum that the first tile then flushes).
cudaError_t launch_encode_segments(const SegQuantArgs& a, const SegmentTable& tab, int bits, int dtype,
                                   unsigned grid, cudaStream_t stream);

struct TileGeom {
    uint64_t elem0;       // flat index of the tile's first element
    uint64_t valid;       // elements from elem0 to the end of the segment
    uint64_t word0;       // code word of the tile's first row
    uint64_t words_end;   // one past the segment's last code word
    uint64_t seg;         // segment index (= index of its scale)
    uint32_t tile_local;  // tile index inside the segment
    int rows;             // rows of this tile that exist
};

template <int BITS>
__device__ __forceinline__ TileGeom locate_tile(const SegmentTable& tab, uint32_t tile)
{
    TileGeom g;
    uint64_t seg_start, seg_len, code0;
    if (tab.uniform_bucket != 0) {
        g.seg = tile / tab.tiles_per_bucket;
        g.tile_local = tile % tab.tiles_per_bucket;
        seg_start = g.seg * tab.uniform_bucket;
        const uint64_t left = tab.n_total - seg_start;
        seg_len = left < tab.uniform_bucket ? left : tab.uniform_bucket;
        code0 = seg_start / 32 * BITS;
    } else {
        int lo = 0, hi = tab.nseg - 1;              // last j with tile_start[j] <= tile
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (tab.tile_start[mid] <= tile) lo = mid; else hi = mid - 1;
        }
        g.seg = (uint64_t)lo;
        g.tile_local = tile - tab.tile_start[lo];
        seg_start = tab.seg_off[lo];
        seg_len = tab.seg_off[lo + 1] - seg_start;
        code0 = tab.code_off[lo];
    }
    const uint64_t done = (uint64_t)g.tile_local * (kMaxTileRows * 32);
    g.elem0 = seg_start + done;
    g.valid = seg_len - done;
    g.word0 = code0 + (uint64_t)g.tile_local * kMaxTileRows * BITS;
    g.words_end = code0 + (seg_len * BITS + 31) / 32;
    const uint64_t rows = (g.valid + 31) / 32;
    g.rows = (int)(rows < (uint64_t)kMaxTileRows ? rows : (uint64_t)kMaxTileRows);
    return g;
}

}  // namespace mqg
