// KV commit (Sec. 4.3 / Algorithm 4 in per-step form): the K/V rows of the accepted path are
// appended, gap-free and in path order, behind each sequence's committed entries.
#include "common.cuh"

namespace reader {

// One CTA per sequence: check that the page table can hold the new positions, copy the rows
// (16-byte chunks, all KV heads), then bump seq_lens.  Nothing is written for a sequence that
// fails the check.
__global__ void __launch_bounds__(256) kv_commit_kernel(__nv_bfloat16 *__restrict__ k_pool,
                                                        __nv_bfloat16 *__restrict__ v_pool, int num_pages, int Hkv,
                                                        int D, const int32_t *__restrict__ page_table, int max_pages,
                                                        int32_t *__restrict__ seq_lens, int shared_prefix_len,
                                                        const __nv_bfloat16 *__restrict__ k_tree,
                                                        const __nv_bfloat16 *__restrict__ v_tree, int T,
                                                        const int32_t *__restrict__ path,
                                                        const int32_t *__restrict__ n_acc, int max_path,
                                                        int update_seq_lens, int32_t *__restrict__ slots,
                                                        int32_t *__restrict__ status) {
    pdl_wait();
    pdl_launch_dependents();
    const int b = blockIdx.x, tid = threadIdx.x;
    __shared__ int ok_s;
    const int L = seq_lens[b];
    const int n = n_acc[b];
    if (tid == 0) ok_s = 1;
    __syncthreads();
    for (int k = tid; k < max_path; k += blockDim.x) slots[(size_t)b * max_path + k] = -1;
    if (n <= 0) {
        if (tid == 0) status[b] = READER_OK;
        return;
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
        if (tid == 0) status[b] = READER_ERR_CAPACITY;
        return;
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
    for (int k = tid; k < n; k += blockDim.x) {
        const int pos = L + k;
        slots[(size_t)b * max_path + k] = page_table[(size_t)b * max_pages + pos / kPage] * kPage + pos % kPage;
    }
    if (tid == 0) {
        status[b] = READER_OK;
        if (update_seq_lens) seq_lens[b] = L + n;
    }
}

void launch_kv_commit(const reader_kv_cache &c, const __nv_bfloat16 *k_tree, const __nv_bfloat16 *v_tree, int B, int T,
                      const int32_t *path, const int32_t *n_acc, int max_path, int update_seq_lens, int32_t *slots,
                      int32_t *status, cudaStream_t st) {
    if (B <= 0) return;
    launch_pdl(kv_commit_kernel, dim3(B), dim3(256), 0, st, reinterpret_cast<__nv_bfloat16 *>(c.k_pool),
                                        reinterpret_cast<__nv_bfloat16 *>(c.v_pool), c.num_pages, c.n_kv_heads,
                                        c.head_dim, c.page_table, c.max_pages_per_seq, c.seq_lens,
                                        c.shared_prefix_len, k_tree, v_tree, T, path, n_acc, max_path,
                                        update_seq_lens, slots, status);
}

}  // namespace reader
