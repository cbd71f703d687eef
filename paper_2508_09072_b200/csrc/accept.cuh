// The acceptance walk of one sequence (Algorithm 5; Appendix C invariants 2-3), shared by the kernels
// that run it: reduce the argmax partials (or take given target ids), find the deepest root path whose
// every non-root node carries the token the target model picks after its parent.
#pragma once
#include <limits.h>

#include "common.cuh"
#include "tree.cuh"

namespace reader {

struct Best {
    float v;
    int i;
};

__device__ __forceinline__ Best better(Best a, Best b) {
    // larger value wins; equal values: lower index.  NaNs never enter (they fail every '>' below).
    if (b.v > a.v || (b.v == a.v && b.i < a.i)) return b;
    return a;
}

// Called by one whole warp for sequence b; par and tgt are that warp's shared-memory scratch of
// kMaxNodes words each.
__device__ __forceinline__ void accept_sequence(int b, int lane, int32_t *par, int32_t *tgt,
                                                const int32_t *__restrict__ parent, const int32_t *__restrict__ tok,
                                                int32_t *__restrict__ target, int T, int max_path,
                                                const float *__restrict__ part_val, const int32_t *__restrict__ part_idx,
                                                int splits, int32_t *__restrict__ path, int32_t *__restrict__ n_acc,
                                                int32_t *__restrict__ bonus, int32_t *__restrict__ status) {
    for (int j = lane; j < T; j += 32) {
        par[j] = parent[(size_t)b * T + j];
        int t;
        if (splits > 0) {
            Best best{-INFINITY, INT_MAX};
            const size_t row = (size_t)b * T + j;
            for (int s = 0; s < splits; ++s) best = better(best, Best{part_val[row * splits + s], part_idx[row * splits + s]});
            t = best.i == INT_MAX ? 0 : best.i;
            target[row] = t;
        } else {
            t = target[(size_t)b * T + j];
        }
        tgt[j] = t;
    }
    __syncwarp();
    const bool valid = warp_tree_valid(par, T, lane);
    for (int k = lane; k < max_path; k += 32) path[(size_t)b * max_path + k] = -1;
    if (!valid) {
        if (lane == 0) { n_acc[b] = 0; bonus[b] = -1; status[b] = READER_ERR_BAD_TREE; }
        return;
    }
    // which nodes carry the token the target model picks after their parent
    uint32_t okw[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int j = lane + 32 * i;
        const bool ok = j < T && (j == 0 || tok[(size_t)b * T + j] == tgt[par[j]]);
        okw[i] = __ballot_sync(0xffffffffu, ok);
    }
    const uint64_t ok_lo = (uint64_t)okw[0] | ((uint64_t)okw[1] << 32);
    const uint64_t ok_hi = (uint64_t)okw[2] | ((uint64_t)okw[3] << 32);

    // a node is accepted iff it and all its ancestors are ok; deepest wins, lowest index among equals
    int key = 0;
    uint64_t my_lo[4], my_hi[4];
    int my_lv[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int j = lane + 32 * i;
        my_lo[i] = my_hi[i] = 0; my_lv[i] = 0;
        if (j < T) {
            node_ancestors(par, T, j, my_lo[i], my_hi[i], my_lv[i]);
            const bool acc = ((my_lo[i] & ~ok_lo) | (my_hi[i] & ~ok_hi)) == 0;
            if (acc && my_lv[i] <= max_path) key = max(key, my_lv[i] * 256 + (255 - j));
        }
    }
    for (int d = 16; d > 0; d >>= 1) key = max(key, __shfl_xor_sync(0xffffffffu, key, d));
    const int end = 255 - (key & 255);
    const int n = key >> 8;
    uint64_t e_lo = 0, e_hi = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i)
        if ((end >> 5) == i) {
            e_lo = __shfl_sync(0xffffffffu, my_lo[i], end & 31);
            e_hi = __shfl_sync(0xffffffffu, my_hi[i], end & 31);
        }
    __syncwarp();   // the -1 fill above is ordered before the path writes below
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int j = lane + 32 * i;
        const bool on = j < 64 ? (e_lo >> j) & 1 : (e_hi >> (j - 64)) & 1;
        if (j < T && on) path[(size_t)b * max_path + my_lv[i] - 1] = j;
    }
    if (lane == 0) { n_acc[b] = n; bonus[b] = tgt[end]; status[b] = READER_OK; }
}

}  // namespace reader
