// KV commit (Sec. 4.3 / Algorithm 4 in per-step form): the K/V rows of the accepted path are
// appended, gap-free and in path order, behind each sequence's committed entries.
#include "kv_commit.cuh"

namespace reader {

// One CTA per sequence; then seq_lens is bumped.
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
    const int b = blockIdx.x;
    const int L = seq_lens[b], n = n_acc[b];
    const bool done = commit_sequence(k_pool, v_pool, num_pages, Hkv, D, page_table, max_pages, L, shared_prefix_len,
                                      k_tree, v_tree, T, path, n, max_path, b, slots, status);
    if (done && update_seq_lens && threadIdx.x == 0) seq_lens[b] = L + n;
}

// All layers of a model in one launch: block (b, l) commits sequence b into layer l's pools.  The
// layers share page table and lengths, so the check has the same outcome in every layer; block (b, 0)
// reports it.  No block writes seq_lens (all of them read it): a second kernel bumps it afterwards.
__global__ void __launch_bounds__(256) kv_commit_layers_kernel(const CommitLayers layers, int layer0, int num_pages,
                                                               int Hkv, int D, const int32_t *__restrict__ page_table,
                                                               int max_pages, const int32_t *__restrict__ seq_lens,
                                                               int shared_prefix_len, int T,
                                                               const int32_t *__restrict__ path,
                                                               const int32_t *__restrict__ n_acc, int max_path,
                                                               int32_t *__restrict__ slots, int32_t *__restrict__ status) {
    pdl_wait();
    pdl_launch_dependents();
    const int b = blockIdx.x, l = blockIdx.y;
    const bool first = layer0 + l == 0;
    commit_sequence(layers.k_pool[l], layers.v_pool[l], num_pages, Hkv, D, page_table, max_pages, seq_lens[b],
                    shared_prefix_len, layers.k_tree[l], layers.v_tree[l], T, path, n_acc[b], max_path, b,
                    first ? slots : nullptr, first ? status : nullptr);
}

__global__ void __launch_bounds__(256) bump_seq_lens_kernel(int32_t *__restrict__ seq_lens, const int32_t *__restrict__ n_acc,
                                                            const int32_t *__restrict__ status, int B) {
    pdl_wait();
    pdl_launch_dependents();
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b < B && status[b] == READER_OK && n_acc[b] > 0) seq_lens[b] += n_acc[b];
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

void launch_kv_commit_layers(const reader_kv_cache &c, const CommitLayers *chunks, int n_layers, int B, int T,
                             const int32_t *path, const int32_t *n_acc, int max_path, int update_seq_lens,
                             int32_t *slots, int32_t *status, cudaStream_t st) {
    if (B <= 0 || n_layers <= 0) return;
    for (int l0 = 0; l0 < n_layers; l0 += kCommitLayersPerLaunch) {
        const int nl = n_layers - l0 < kCommitLayersPerLaunch ? n_layers - l0 : kCommitLayersPerLaunch;
        launch_pdl(kv_commit_layers_kernel, dim3(B, nl), dim3(256), 0, st, chunks[l0 / kCommitLayersPerLaunch], l0,
                   c.num_pages, c.n_kv_heads, c.head_dim, c.page_table, c.max_pages_per_seq,
                   static_cast<const int32_t *>(c.seq_lens), c.shared_prefix_len, T, path, n_acc, max_path, slots, status);
    }
    if (update_seq_lens)
        launch_pdl(bump_seq_lens_kernel, dim3((B + 255) / 256), dim3(256), 0, st, c.seq_lens, n_acc,
                   static_cast<const int32_t *>(status), B);
}

}  // namespace reader
