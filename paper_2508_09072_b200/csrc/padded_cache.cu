// The padded batch cache of Sec. 4.3 kept as a cache: how it grows in a step, and the bookkeeping of
// its common length.  (Its attention runs through the same kernels as the paged cache, see
// AttnParams::valid_bits; its compaction is kv_rearrange.cu.)
//
// Growth: every sample's row grows by the batch's longest accepted span; a sample that accepted less
// gets zero rows marked as padding for the difference -- the transient footprint the paper describes.
// k, v [B][Hkv][cap][D]; valid [B][cap]; *extent the common length.
#include "common.cuh"

namespace reader {

// Block-wide, same answer in every block: by how many rows the cache grows and whether the step can
// be applied at all (all or nothing, because the length is common to the batch).
__device__ __forceinline__ bool append_plan(const int32_t *__restrict__ path, const int32_t *__restrict__ n_acc, int B,
                                            int T, int max_path, int cap, int extent, int &grow) {
    __shared__ int s_grow, s_bad;
    if (threadIdx.x == 0) {
        s_grow = 0;
        s_bad = 0;
    }
    __syncthreads();
    int g = 0, bad = 0;
    for (int i = threadIdx.x; i < B * max_path; i += blockDim.x) {
        const int b = i / max_path, k = i - b * max_path;
        const int n = n_acc[b];
        if (n < 0 || n > max_path) {
            bad = 1;
        } else {
            g = max(g, n);
            if (k < n) {
                const int node = path[i];
                if (node < 0 || node >= T) bad = 1;
            }
        }
    }
    if (g > 0) atomicMax(&s_grow, g);
    if (bad) atomicOr(&s_bad, 1);
    __syncthreads();
    grow = s_grow;
    return !s_bad && extent >= 0 && extent <= cap && (int64_t)extent + grow <= (int64_t)cap;
}

// Block (b, h): the accepted rows of KV head h of sample b behind the common length, then zero rows.
__global__ void __launch_bounds__(256) padded_append_kernel(__nv_bfloat16 *__restrict__ k, __nv_bfloat16 *__restrict__ v,
                                                            int B, int Hkv, int cap, int D, uint8_t *__restrict__ valid,
                                                            const int32_t *__restrict__ extent,
                                                            const __nv_bfloat16 *__restrict__ k_tree,
                                                            const __nv_bfloat16 *__restrict__ v_tree, int T,
                                                            const int32_t *__restrict__ path,
                                                            const int32_t *__restrict__ n_acc, int max_path,
                                                            int32_t *__restrict__ status) {
    pdl_wait();
    pdl_launch_dependents();
    const int b = blockIdx.x, h = blockIdx.y, tid = threadIdx.x;
    const int E = *extent;
    int grow = 0;
    const bool ok = append_plan(path, n_acc, B, T, max_path, cap, E, grow);
    if (h == 0 && tid == 0) status[b] = ok ? READER_OK : READER_ERR_CAPACITY;
    if (!ok) return;
    const int n = n_acc[b];
    const int ppr = D / 8;   // 16-byte pieces per row
    const size_t row0 = ((size_t)b * Hkv + h) * cap + E;
    for (int i = tid; i < 2 * grow * ppr; i += blockDim.x) {
        const int which = i / (grow * ppr), rest = i - which * grow * ppr;
        const int r = rest / ppr, piece = rest - r * ppr;
        uint4 x = make_uint4(0, 0, 0, 0);
        if (r < n) {
            const size_t src = (((size_t)b * T + path[(size_t)b * max_path + r]) * Hkv + h) * D;
            x = reinterpret_cast<const uint4 *>((which ? v_tree : k_tree) + src)[piece];
        }
        reinterpret_cast<uint4 *>((which ? v : k) + (row0 + r) * D)[piece] = x;
    }
    if (h == 0)
        for (int r = tid; r < grow; r += blockDim.x) valid[(size_t)b * cap + E + r] = r < n;
}

// After every block of the kernel above has read the common length: move it.
__global__ void __launch_bounds__(256) padded_extent_kernel(int B, int cap, int32_t *__restrict__ extent, int T,
                                                            const int32_t *__restrict__ path,
                                                            const int32_t *__restrict__ n_acc, int max_path) {
    pdl_wait();
    pdl_launch_dependents();
    const int E = *extent;
    int grow = 0;
    const bool ok = append_plan(path, n_acc, B, T, max_path, cap, E, grow);
    if (ok && threadIdx.x == 0) *extent = E + grow;
}

// *extent = the longest of the compacted rows.
__global__ void __launch_bounds__(256) set_extent_kernel(const int32_t *__restrict__ lengths, int B,
                                                         int32_t *__restrict__ extent) {
    pdl_wait();
    pdl_launch_dependents();
    __shared__ int s_max;
    if (threadIdx.x == 0) s_max = 0;
    __syncthreads();
    int m = 0;
    for (int b = threadIdx.x; b < B; b += blockDim.x) m = max(m, lengths[b]);
    if (m > 0) atomicMax(&s_max, m);
    __syncthreads();
    if (threadIdx.x == 0) *extent = s_max;
}

void launch_padded_append(__nv_bfloat16 *k, __nv_bfloat16 *v, int B, int Hkv, int cap, int D, uint8_t *valid,
                          int32_t *extent, const __nv_bfloat16 *k_tree, const __nv_bfloat16 *v_tree, int T,
                          const int32_t *path, const int32_t *n_acc, int max_path, int32_t *status, cudaStream_t st) {
    if (B <= 0) return;
    launch_pdl(padded_append_kernel, dim3(B, Hkv), dim3(256), 0, st, k, v, B, Hkv, cap, D, valid, extent, k_tree, v_tree, T,
               path, n_acc, max_path, status);
    launch_pdl(padded_extent_kernel, dim3(1), dim3(256), 0, st, B, cap, extent, T, path, n_acc, max_path);
}

void launch_set_extent(const int32_t *lengths, int B, int32_t *extent, cudaStream_t st) {
    if (B <= 0) return;
    launch_pdl(set_extent_kernel, dim3(1), dim3(256), 0, st, lengths, B, extent);
}

}  // namespace reader
