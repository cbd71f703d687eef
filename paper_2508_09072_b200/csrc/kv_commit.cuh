// The per-sequence commit (Sec. 4.3 / Algorithm 4 in per-step form), shared by the kernels that run it.
#pragma once
#include "common.cuh"

namespace reader {

// The commit of one sequence into one layer's pools, by one CTA: check that the page table can hold
// the new positions, copy the rows (16-byte chunks, all KV heads).  Nothing is written for a sequence
// that fails the check.  slots / status may be null (layers other than the first do not repeat them).
// Returns whether rows were committed (the same value in every thread).
__device__ __forceinline__ bool commit_sequence(__nv_bfloat16 *__restrict__ k_pool, __nv_bfloat16 *__restrict__ v_pool,
                                                int num_pages, int Hkv, int D, const int32_t *__restrict__ page_table,
                                                int max_pages, int L, int shared_prefix_len,
                                                const __nv_bfloat16 *__restrict__ k_tree,
                                                const __nv_bfloat16 *__restrict__ v_tree, int T,
                                                const int32_t *path /* may have been written earlier in the same kernel */, int n, int max_path, int b,
                                                int32_t *__restrict__ slots, int32_t *__restrict__ status) {
    const int tid = threadIdx.x;
    __shared__ int ok_s;
    if (tid == 0) ok_s = 1;
    __syncthreads();
    if (slots)
        for (int k = tid; k < max_path; k += blockDim.x) slots[(size_t)b * max_path + k] = -1;
    if (n <= 0) {
        if (tid == 0 && status) status[b] = READER_OK;
        return false;
    }
    bool ok = n <= max_path && L >= 0 && L >= shared_prefix_len && (int64_t)L + n <= (int64_t)max_pages * kPage;
    if (ok)
        for (int k = tid; k < n; k += blockDim.x) {
            const int pg = page_table[(size_t)b * max_pages + (L + k) / kPage];
            const int node = path[(size_t)b * max_path + k];
            if (pg < 0 || pg >= num_pages || node < 0 || node >= T) ok = false;
        }
    if (!ok) ok_s = 0;
    __syncthreads();
    if (!ok_s) {
        if (tid == 0 && status) status[b] = READER_ERR_CAPACITY;
        return false;
    }
    const int chunks_per_head = D / 8;                  // 16-byte chunks per (node, head) row
    const int chunks_per_node = Hkv * chunks_per_head;
    for (int c = tid; c < n * chunks_per_node; c += blockDim.x) {
        const int k = c / chunks_per_node;
        const int r = c - k * chunks_per_node;
        const int h = r / chunks_per_head, x = r - h * chunks_per_head;
        const int pos = L + k;
        const int pg = page_table[(size_t)b * max_pages + pos / kPage];
        const int node = path[(size_t)b * max_path + k];
        const size_t src = (((size_t)b * T + node) * Hkv + h) * D + x * 8;
        const size_t dst = (((size_t)pg * Hkv + h) * kPage + pos % kPage) * D + x * 8;
        *reinterpret_cast<uint4 *>(k_pool + dst) = *reinterpret_cast<const uint4 *>(k_tree + src);
        *reinterpret_cast<uint4 *>(v_pool + dst) = *reinterpret_cast<const uint4 *>(v_tree + src);
    }
    if (slots)
        for (int k = tid; k < n; k += blockDim.x) {
            const int pos = L + k;
            slots[(size_t)b * max_path + k] = page_table[(size_t)b * max_pages + pos / kPage] * kPage + pos % kPage;
        }
    if (tid == 0 && status) status[b] = READER_OK;
    return true;
}

}  // namespace reader
