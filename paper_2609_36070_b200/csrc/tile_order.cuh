// Static tile order of the persistent 128-row-tile GEMM kernels (bf16 and MXFP8).
#pragma once
#include "mok_internal.cuh"

namespace mok {
namespace tc {

constexpr int GROUP_ROWS = 2048;               // rows of one rasterisation group (16 tiles of 128 rows)

struct Tile { int row0, n, e, m; };   // row0: first row of the (pair) tile in the padded row space

// Tile L of the static schedule.  `tm` = rows per tile (128 x CTAS).  Inside an expert, M tiles are taken in groups
// of GROUP_ROWS rows: all N tiles of a group before the next group, M fastest, so the group's activations stay in
// L2 while the expert's weight tiles stream.
__device__ __forceinline__ Tile decode_tile(const GemmArgs& a, int L, int n_nt, int n_mt_total, int tm) {
    Tile t;
    int mt0, m_cnt, pad0;
    if (a.dense_rows > 0) {
        t.e = 0; mt0 = 0; m_cnt = n_mt_total; pad0 = 0;
    } else {
        t.e = __ldg(a.tile_expert + L / n_nt);
        mt0 = __ldg(a.mt_start + t.e);
        m_cnt = __ldg(a.mt_start + t.e + 1) - mt0;
        pad0 = __ldg(a.pad_offsets + t.e);
    }
    const int group_m = GROUP_ROWS / tm;
    const int r = L - n_nt * mt0;
    const int per_group = group_m * n_nt;
    const int g = r / per_group;
    const int rem = r - g * per_group;
    const int in_group = min(group_m, m_cnt - g * group_m);
    t.n = rem / in_group;
    t.m = g * group_m + (rem - t.n * in_group);
    // first row in the padded row space: the expert's segment start (a multiple of the padding granularity, which
    // may be finer than the tile: 256-row pair tiles over 128-row padding) plus whole tiles
    t.row0 = pad0 + t.m * tm;
    return t;
}

}  // namespace tc
}  // namespace mok
