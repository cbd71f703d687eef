// KVCacheRearrange (Sec. 4.3, Algorithm 4) on the paper's own cache layout: a rectangular batch
// cache k, v [B][Hkv][cap][D] whose rows hold real entries and internal padding, told apart by a
// validity mask [B][cap].  Per sample the real entries are moved to the front in order, the tail is
// zeroed, the mask becomes 1..10..0 and the number of entries is reported.
//
// One block per (sample, KV head, K or V) walks its cap positions in chunks of up to 256 rows (as many
// as fit 40 KB of shared memory: 160 at head_dim 128): the chunk's mask bytes are prefix-summed, its real
// rows are staged in shared memory at their compacted places and then written to positions that never
// lie beyond the chunk's own end -- everything a write can overwrite has been read already, so the
// compaction is in place.  A chunk that is already where it belongs is not touched.  A second kernel
// rewrites the mask once every block is done with it.
#include "common.cuh"

namespace reader {

constexpr int kMaxChunkRows = 256;            // one mask ballot per warp of the 256-thread block
constexpr int kStageBytes = 40 * 1024;     // dynamic; with the static arrays below still within the 48 KB a kernel gets by default

__global__ void __launch_bounds__(256) rearrange_rows_kernel(__nv_bfloat16 *__restrict__ k, __nv_bfloat16 *__restrict__ v,
                                                             int Hkv, int cap, int D, int chunk_rows,
                                                             const uint8_t *__restrict__ valid) {
    pdl_wait();
    pdl_launch_dependents();
    extern __shared__ __align__(16) unsigned char stage[];   // chunk_rows rows of D bf16
    __shared__ int dest[kMaxChunkRows];                       // compacted place within the chunk, or -1
    __shared__ unsigned bal_s[8];
    const int bh = blockIdx.x, b = bh / Hkv;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    __nv_bfloat16 *base = (blockIdx.y == 0 ? k : v) + (size_t)bh * cap * D;
    const uint8_t *mask = valid + (size_t)b * cap;
    const int pieces_per_row = D / 8;                         // 16-byte pieces
    uint4 *stage4 = reinterpret_cast<uint4 *>(stage);

    int done = 0;                                             // entries already in place in front
    for (int c0 = 0; c0 < cap; c0 += chunk_rows) {
        const int rows = min(chunk_rows, cap - c0);
        {                                                     // 32 mask bytes per warp -> one ballot each
            const int r = warp * 32 + lane;
            const unsigned bal = __ballot_sync(0xffffffffu, r < rows && mask[c0 + r] != 0);
            if (lane == 0) bal_s[warp] = bal;
        }
        __syncthreads();
        int count = 0, before = 0;                            // real rows in the chunk / in the warps before this one
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const int n = __popc(bal_s[q]);
            count += n;
            if (q < warp) before += n;
        }
        {                                                     // place of every real row among the chunk's real rows
            const bool real = (bal_s[warp] >> lane) & 1u;
            dest[warp * 32 + lane] = real ? before + __popc(bal_s[warp] & ((1u << lane) - 1)) : -1;
        }
        __syncthreads();
        const bool in_place = done == c0 && count == rows;    // nothing before it was dropped and nothing in it is
        if (!in_place && count > 0) {
            // eight 16-byte loads per thread in flight before the first of them is put down (one at a time, each
            // waited for before the next was issued, the pass ran at 3.0 TB/s whatever the chunk size)
            constexpr int kInFlight = 8;
            const int total = rows * pieces_per_row;
            for (int i0 = tid; i0 < total; i0 += kInFlight * blockDim.x) {
                uint4 val[kInFlight];
                int at[kInFlight];
#pragma unroll
                for (int q = 0; q < kInFlight; ++q) {
                    const int i = i0 + q * blockDim.x;
                    at[q] = -1;
                    if (i < total) {
                        const int r = i / pieces_per_row, piece = i - r * pieces_per_row;
                        const int d = dest[r];
                        if (d >= 0) {
                            at[q] = d * pieces_per_row + piece;
                            val[q] = reinterpret_cast<const uint4 *>(base + (size_t)(c0 + r) * D)[piece];
                        }
                    }
                }
#pragma unroll
                for (int q = 0; q < kInFlight; ++q)
                    if (at[q] >= 0) stage4[at[q]] = val[q];
            }
            __syncthreads();                                   // the whole chunk is read before any of it is overwritten
            uint4 *out = reinterpret_cast<uint4 *>(base + (size_t)done * D);
            for (int i = tid; i < count * pieces_per_row; i += blockDim.x) out[i] = stage4[i];
        }
        done += count;
        __syncthreads();                                       // stage, dest and the ballots are reused
    }
    // the vacated tail
    uint4 *tail = reinterpret_cast<uint4 *>(base + (size_t)done * D);
    for (size_t i = tid; i < (size_t)(cap - done) * pieces_per_row; i += blockDim.x) tail[i] = make_uint4(0, 0, 0, 0);
}

__global__ void __launch_bounds__(256) rearrange_mask_kernel(uint8_t *__restrict__ valid, int cap,
                                                             int32_t *__restrict__ lengths) {
    pdl_wait();
    pdl_launch_dependents();
    __shared__ int total;
    const int b = blockIdx.x;
    uint8_t *mask = valid + (size_t)b * cap;
    if (threadIdx.x == 0) total = 0;
    __syncthreads();
    int n = 0;
    for (int t = threadIdx.x; t < cap; t += blockDim.x) n += mask[t] != 0;
    for (int d = 16; d > 0; d >>= 1) n += __shfl_xor_sync(0xffffffffu, n, d);
    if ((threadIdx.x & 31) == 0) atomicAdd(&total, n);
    __syncthreads();
    n = total;
    for (int t = threadIdx.x; t < cap; t += blockDim.x) mask[t] = t < n;
    if (threadIdx.x == 0) lengths[b] = n;
}

void launch_kv_rearrange(__nv_bfloat16 *k, __nv_bfloat16 *v, int B, int Hkv, int cap, int D, uint8_t *valid,
                         int32_t *lengths, cudaStream_t st) {
    if (B <= 0) return;
    int chunk_rows = kStageBytes / (D * 2) / 32 * 32;
    if (chunk_rows > kMaxChunkRows) chunk_rows = kMaxChunkRows;
    launch_pdl(rearrange_rows_kernel, dim3(B * Hkv, 2), dim3(256), (size_t)chunk_rows * D * 2, st, k, v, Hkv, cap, D, chunk_rows, valid);
    launch_pdl(rearrange_mask_kernel, dim3(B), dim3(256), 0, st, valid, cap, lengths);
}

}  // namespace reader
