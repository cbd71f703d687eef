// Acceptance (Algorithm 5; Appendix C invariants 2-3 with the greedy policy): row argmax
// of the target logits with a lowest-index tie-break, then the longest root path whose every
// non-root node carries the token the target model picks after its parent.
#include "accept.cuh"

namespace reader {

// grid (rows, splits): block (r, s) scans columns [s*chunk, min(V, (s+1)*chunk)) of row r.
template <bool kVec>
__global__ void __launch_bounds__(256) argmax_kernel(const float *__restrict__ logits, int64_t vocab, int chunk,
                                                     int splits, float *__restrict__ part_val,
                                                     int32_t *__restrict__ part_idx) {
    pdl_wait();
    pdl_launch_dependents();
    const int64_t row = blockIdx.x;
    const int split = blockIdx.y;
    const int c0 = split * chunk;
    const int c1 = (int)min((int64_t)c0 + chunk, vocab);
    const float *src = logits + row * vocab;
    Best best{-INFINITY, INT_MAX};
    if (kVec) {
        const float4 *v4 = reinterpret_cast<const float4 *>(src + c0);
        const int n4 = (c1 - c0) >> 2;
        int i = threadIdx.x;
        for (; i + 7 * 256 < n4; i += 8 * 256) {
            float4 a[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) a[u] = __ldcs(v4 + i + u * 256);
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int at = c0 + 4 * (i + u * 256);
                if (a[u].x > best.v) { best.v = a[u].x; best.i = at; }
                if (a[u].y > best.v) { best.v = a[u].y; best.i = at + 1; }
                if (a[u].z > best.v) { best.v = a[u].z; best.i = at + 2; }
                if (a[u].w > best.v) { best.v = a[u].w; best.i = at + 3; }
            }
        }
        for (; i < n4; i += 256) {
            const float4 a = __ldcs(v4 + i);
            const int at = c0 + 4 * i;
            if (a.x > best.v) { best.v = a.x; best.i = at; }
            if (a.y > best.v) { best.v = a.y; best.i = at + 1; }
            if (a.z > best.v) { best.v = a.z; best.i = at + 2; }
            if (a.w > best.v) { best.v = a.w; best.i = at + 3; }
        }
        for (int c = c0 + 4 * n4 + threadIdx.x; c < c1; c += 256) {
            const float a = src[c];
            if (a > best.v) { best.v = a; best.i = c; }
        }
    } else {
        for (int c = c0 + threadIdx.x; c < c1; c += 256) {
            const float a = src[c];
            if (a > best.v) { best.v = a; best.i = c; }
        }
    }
    for (int d = 16; d > 0; d >>= 1) {
        Best o{__shfl_xor_sync(0xffffffffu, best.v, d), __shfl_xor_sync(0xffffffffu, best.i, d)};
        best = better(best, o);
    }
    __shared__ Best wb[8];
    if ((threadIdx.x & 31) == 0) wb[threadIdx.x >> 5] = best;
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int k = 1; k < 8; ++k) best = better(best, wb[k]);
        part_val[row * splits + split] = best.v;
        part_idx[row * splits + split] = best.i;
    }
}

void launch_argmax(const float *logits, int64_t rows, int64_t vocab, int splits, float *part_val,
                   int32_t *part_idx, cudaStream_t st) {
    if (rows <= 0) return;
    int chunk = (int)((vocab + splits - 1) / splits);
    chunk = (chunk + 3) & ~3;
    dim3 grid((unsigned)rows, (unsigned)splits);
    if (vocab % 4 == 0)
        launch_pdl(argmax_kernel<true>, grid, dim3(256), 0, st, logits, vocab, chunk, splits, part_val, part_idx);
    else
        launch_pdl(argmax_kernel<false>, grid, dim3(256), 0, st, logits, vocab, chunk, splits, part_val, part_idx);
}

// One warp per sequence.
__global__ void __launch_bounds__(128) accept_kernel(const int32_t *__restrict__ parent,
                                                     const int32_t *__restrict__ tok, int32_t *__restrict__ target,
                                                     int B, int T, int max_path, const float *__restrict__ part_val,
                                                     const int32_t *__restrict__ part_idx, int splits,
                                                     int32_t *__restrict__ path, int32_t *__restrict__ n_acc,
                                                     int32_t *__restrict__ bonus, int32_t *__restrict__ status) {
    __shared__ int32_t par_s[4][kMaxNodes];
    __shared__ int32_t tgt_s[4][kMaxNodes];
    pdl_wait();
    pdl_launch_dependents();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int b = blockIdx.x * 4 + warp;
    if (b >= B) return;
    accept_sequence(b, lane, par_s[warp], tgt_s[warp], parent, tok, target, T, max_path, part_val, part_idx, splits, path,
                    n_acc, bonus, status);
}

void launch_accept(const int32_t *parent, const int32_t *tok, int32_t *target, int B, int T, int max_path,
                   const float *part_val, const int32_t *part_idx, int splits, int32_t *path, int32_t *n_acc,
                   int32_t *bonus, int32_t *status, cudaStream_t st) {
    if (B <= 0) return;
    launch_pdl(accept_kernel, dim3((B + 3) / 4), dim3(128), 0, st, parent, tok, target, B, T, max_path, part_val, part_idx, splits,
                                               path, n_acc, bonus, status);
}

}  // namespace reader
