// Row plan of the channel-compacted FFN.  Rows of absent-modality tokens are
// skipped and samples may use different kept-channel lists, so the present
// rows are regrouped: per list, the present rows of its samples (sample order,
// token order) form one row sequence that is cut into tiles of `tile_rows`.
// A tile therefore uses one weight set and is full except for the last tile
// of each list.  The plan is a flat table of global row indices (b*T + t),
// list after list, plus the per-list offsets into it.
#pragma once
#include "common.cuh"

struct FfnPlan {
    // all device pointers into the workspace
    int32_t* sample_row0;   // [B]          offset in rowidx of sample b's first present row
    int32_t* list_row0;     // [n_lists+1]  offset in rowidx of each list's rows
    int32_t* tile_start;    // [n_lists+1]  first tile of each list; [n_lists] = total tiles
    int32_t* rowidx;        // [B*T]        global row (b*T + t) of every present row, list-major
    int32_t* rowout;        // same shape or null: row of Y a result goes to, if not the row of X it came from
                            //              (Sparse-MoE: X row = token, Y row = (token, routing slot))
};

// The fused pair alone, on a row plan and materialised weights that are already in place.
int launch_ffn_main(sentry_ctx* ctx, const FfnArgs& a, const FfnPlan& plan, void* w1p, void* w2p, int kc_pad,
                    int max_tiles, cudaStream_t st);

#ifdef __CUDACC__
// Locate tile `tile` -> list l, offset of its first row in rowidx, and its row count;
// returns false if the tile is past the end.
__device__ __forceinline__ bool ffn_tile_lookup(const FfnPlan& p, int n_lists, int tile,
                                                int tile_rows, int& l, int& row0, int& n_rows) {
    if (tile >= p.tile_start[n_lists]) return false;
    l = 0;
    while (l + 1 < n_lists && p.tile_start[l + 1] <= tile) ++l;
    const int slot0 = (tile - p.tile_start[l]) * tile_rows;
    row0 = p.list_row0[l] + slot0;
    n_rows = min(tile_rows, p.list_row0[l + 1] - row0);
    return true;
}
#endif
