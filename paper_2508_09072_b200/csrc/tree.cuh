// Warp-level helpers on a parent array held in shared memory (tree convention: node 0 is the
// root, parent[0] = -1, 0 <= parent[j] < j).
#pragma once
#include "common.cuh"

namespace reader {

// One warp encodes one tree held in shared memory.  Returns (warp-uniform) whether the parent
// array obeys the convention parent[0] = -1, 0 <= parent[j] < j.  On a valid tree every lane
// walks the parent chain of its nodes (j = lane, lane+32, ...); the chain strictly decreases, so
// it ends within T steps.
__device__ __forceinline__ bool warp_tree_valid(const int32_t *par, int T, int lane) {
    bool ok = true;
    for (int j = lane; j < T; j += 32) {
        int p = par[j];
        ok = ok && (j == 0 ? p == -1 : (p >= 0 && p < j));
    }
    return __all_sync(0xffffffffu, ok);
}

__device__ __forceinline__ void node_ancestors(const int32_t *par, int T, int j, uint64_t &lo, uint64_t &hi,
                                               int &level) {
    lo = 0; hi = 0; level = 0;
    int i = j;
    for (int step = 0; step < T && i >= 0; ++step) {
        if (i < 64) lo |= 1ull << i; else hi |= 1ull << (i - 64);
        ++level;
        i = par[i];
    }
}

}  // namespace reader
