// Row plan of the channel-compacted FFN.  Rows of absent-modality tokens are
// skipped and samples may use different kept-channel lists, so the present
// rows are regrouped: per list, the present rows of its samples (sample order,
// token order) form one virtual row sequence that is cut into tiles of
// `tile_rows`.  A tile therefore uses one weight set and is full except for the
// last tile of each list.
#pragma once
#include "common.cuh"

struct FfnPlan {
    // inputs of the main kernels (all device pointers into the workspace)
    uint16_t* vlist;        // [B, T]   present tokens of each sample, ascending
    int32_t* tv;            // [B]      number of present tokens
    int32_t* order;         // [B]      samples sorted by list (stable)
    int32_t* row_prefix;    // [B]      rows of the same list before order[i]
    int32_t* list_start;    // [n_lists+1] segment of `order` per list
    int32_t* list_rows;     // [n_lists]   present rows per list
    int32_t* tile_start;    // [n_lists+1] first tile of each list; [n_lists] = total tiles
};

#ifdef __CUDACC__
// Locate tile `tile` -> list l and first row slot; returns false if past the end.
__device__ __forceinline__ bool ffn_tile_lookup(const FfnPlan& p, int n_lists, int tile,
                                                int tile_rows, int& l, int& slot0, int& n_rows) {
    if (tile >= p.tile_start[n_lists]) return false;
    l = 0;
    while (l + 1 < n_lists && p.tile_start[l + 1] <= tile) ++l;
    slot0 = (tile - p.tile_start[l]) * tile_rows;
    n_rows = min(tile_rows, p.list_rows[l] - slot0);
    return true;
}

// Row slot of list l -> global row index b*T + t.
__device__ __forceinline__ long long ffn_row_of_slot(const FfnPlan& p, int l, int slot, int T) {
    int lo = p.list_start[l], hi = p.list_start[l + 1] - 1;
    while (lo < hi) {  // largest i with row_prefix[i] <= slot
        const int mid = (lo + hi + 1) >> 1;
        if (p.row_prefix[mid] <= slot) lo = mid; else hi = mid - 1;
    }
    const int b = p.order[lo];
    const int t = p.vlist[(size_t)b * T + (slot - p.row_prefix[lo])];
    return (long long)b * T + t;
}
#endif
