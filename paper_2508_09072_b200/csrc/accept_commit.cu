// Acceptance walk and KV commit of a step in one launch (Algorithm 5 followed by Algorithm 4 in
// per-step form): block b finds sequence b's accepted path with its first warp and then, as a whole
// block, appends that path's K/V rows to the sequence's cache.  Same results as accept_kernel
// followed by kv_commit_kernel; one dependent launch fewer per decoding step.
#include "accept.cuh"
#include "kv_commit.cuh"

namespace reader {

__global__ void __launch_bounds__(256) accept_commit_kernel(const int32_t *__restrict__ parent, const int32_t *__restrict__ tok,
                                                            int32_t *__restrict__ target, int T, int max_path,
                                                            const float *__restrict__ part_val,
                                                            const int32_t *__restrict__ part_idx, int splits,
                                                            int32_t *__restrict__ path, int32_t *__restrict__ n_acc,
                                                            int32_t *__restrict__ bonus, int32_t *__restrict__ status,
                                                            __nv_bfloat16 *__restrict__ k_pool, __nv_bfloat16 *__restrict__ v_pool,
                                                            int num_pages, int Hkv, int D,
                                                            const int32_t *__restrict__ page_table, int max_pages,
                                                            int32_t *__restrict__ seq_lens, int shared_prefix_len,
                                                            const __nv_bfloat16 *__restrict__ k_tree,
                                                            const __nv_bfloat16 *__restrict__ v_tree, int update_seq_lens,
                                                            int32_t *__restrict__ slots, int32_t *__restrict__ commit_status) {
    __shared__ int32_t par_s[kMaxNodes];
    __shared__ int32_t tgt_s[kMaxNodes];
    pdl_wait();
    pdl_launch_dependents();
    const int b = blockIdx.x;
    if (threadIdx.x < 32)
        accept_sequence(b, threadIdx.x, par_s, tgt_s, parent, tok, target, T, max_path, part_val, part_idx, splits, path, n_acc,
                        bonus, status);
    __syncthreads();   // the path and its length, written by the first warp, are read by the whole block below
    const int L = seq_lens[b];
    const int n = *reinterpret_cast<volatile const int32_t *>(n_acc + b);
    const bool done = commit_sequence(k_pool, v_pool, num_pages, Hkv, D, page_table, max_pages, L, shared_prefix_len, k_tree,
                                      v_tree, T, path, n, max_path, b, slots, commit_status);
    if (done && update_seq_lens && threadIdx.x == 0) seq_lens[b] = L + n;
}

void launch_accept_commit(const int32_t *parent, const int32_t *tok, int32_t *target, int B, int T, int max_path,
                          const float *part_val, const int32_t *part_idx, int splits, int32_t *path, int32_t *n_acc,
                          int32_t *bonus, int32_t *status, const reader_kv_cache &c, const __nv_bfloat16 *k_tree,
                          const __nv_bfloat16 *v_tree, int update_seq_lens, int32_t *slots, int32_t *commit_status,
                          cudaStream_t st) {
    if (B <= 0) return;
    launch_pdl(accept_commit_kernel, dim3(B), dim3(256), 0, st, parent, tok, target, T, max_path, part_val, part_idx, splits,
               path, n_acc, bonus, status, reinterpret_cast<__nv_bfloat16 *>(c.k_pool), reinterpret_cast<__nv_bfloat16 *>(c.v_pool),
               c.num_pages, c.n_kv_heads, c.head_dim, c.page_table, c.max_pages_per_seq, c.seq_lens, c.shared_prefix_len,
               k_tree, v_tree, update_seq_lens, slots, commit_status);
}

}  // namespace reader
