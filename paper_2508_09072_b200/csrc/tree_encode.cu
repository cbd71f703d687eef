// Tree-mask encoder (Sec. 3.2: M_ij = 1 iff node i is an ancestor of node j, made reflexive) and
// the per-call preparation kernel that validates every sequence and lays out the split-KV work.
#include "common.cuh"
#include "tree.cuh"

namespace reader {

__global__ void __launch_bounds__(128) tree_encode_kernel(const int32_t *__restrict__ parent, int B, int T,
                                                          uint64_t *__restrict__ anc, int32_t *__restrict__ level,
                                                          int32_t *__restrict__ status) {
    __shared__ int32_t par[4][kMaxNodes];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int b = blockIdx.x * 4 + warp;
    if (b >= B) return;
    for (int j = lane; j < T; j += 32) par[warp][j] = parent[(size_t)b * T + j];
    __syncwarp();
    const bool ok = warp_tree_valid(par[warp], T, lane);
    for (int j = lane; j < T; j += 32) {
        uint64_t lo = 0, hi = 0;
        int lv = 0;
        if (ok) node_ancestors(par[warp], T, j, lo, hi, lv);
        anc[((size_t)b * T + j) * 2 + 0] = lo;
        anc[((size_t)b * T + j) * 2 + 1] = hi;
        if (level) level[(size_t)b * T + j] = lv;
    }
    if (lane == 0) status[b] = ok ? READER_OK : READER_ERR_BAD_TREE;
}

void launch_tree_encode(const int32_t *parent, int B, int T, uint64_t *anc, int32_t *level,
                        int32_t *status, cudaStream_t st) {
    if (B <= 0) return;
    tree_encode_kernel<<<(B + 3) / 4, 128, 0, st>>>(parent, B, T, anc, level, status);
}

// One CTA.  Each warp takes sequences b = warp, warp + 32, ...: checks the tree (encoding the
// masks when asked), the committed length against the page table's capacity and every page id
// in use; then warp 0 turns the per-sequence tile counts into the flat prefix the attention
// kernels cut into CTA ranges.  With the padded batch cache (pd.valid != nullptr) there is no page
// table: every sample has the common extent as its length, and the validity bytes below it are packed
// into one 64-bit word per tile for the attention kernels.
__global__ void __launch_bounds__(1024) prepare_kernel(const PaddedIn pd,
                                                       const int32_t *__restrict__ page_table,
                                                       const int32_t *__restrict__ seq_lens, int max_pages,
                                                       int num_pages, const int32_t *__restrict__ parent, int B,
                                                       int T, int n_tree_tiles, int units_per_seq,
                                                       uint64_t *__restrict__ anc_out,
                                                       int32_t *__restrict__ seq_tile_start,
                                                       int32_t *__restrict__ seq_ntiles,
                                                       int32_t *__restrict__ seq_npages,
                                                       int32_t *__restrict__ status,
                                                       int32_t *__restrict__ error_flag,
                                                       __nv_bfloat16 *__restrict__ out, float *__restrict__ lse,
                                                       int Hq, int D) {
    __shared__ int32_t par[32][kMaxNodes];
    __shared__ int s_last;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // A large batch is shared by several blocks, 32 sequences (one per warp) at a time each; the block that
    // finishes last (a counter in the workspace, zeroed by the host before the launch) makes the prefix sums.
    const int gwarp = blockIdx.x * 32 + warp, n_gwarps = gridDim.x * 32;
    pdl_launch_dependents();   // the attention kernel may set itself up meanwhile
    pdl_wait();                // this kernel itself is launched ahead of its predecessor's end
    if (blockIdx.x == 0 && threadIdx.x == 0) *error_flag = 0;
    const bool padded = pd.valid != nullptr;
    const int extent = padded ? *pd.extent : 0;
    const bool extent_ok = extent >= 0 && extent <= pd.cap;
    if (padded && extent_ok) {
        // 16 mask bytes -> 16 bits; pieces from the extent on (up to the end of its tile) read as zero
        const int pieces = ((extent + kPage - 1) / kPage) * (kPage / 16);
        const bool vec = (pd.cap % 16 == 0) && (reinterpret_cast<uintptr_t>(pd.valid) % 16 == 0);
        for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < B * pieces; i += gridDim.x * blockDim.x) {
            const int b = i / pieces, c = i - b * pieces;
            const int first = c * 16, n = min(16, extent - first);   // n <= 0: past the extent
            uint32_t bits = 0;
            if (n > 0) {
                const uint8_t *src = pd.valid + (size_t)b * pd.cap + first;
                if (vec) {
                    const uint4 x = *reinterpret_cast<const uint4 *>(src);
                    const uint32_t w4[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const uint32_t m = __vcmpne4(w4[q], 0u) & 0x08040201u;
                        bits |= ((m | (m >> 8) | (m >> 16) | (m >> 24)) & 0xfu) << (4 * q);
                    }
                } else {
                    for (int r = 0; r < n; ++r) bits |= (src[r] != 0 ? 1u : 0u) << r;
                }
                if (n < 16) bits &= (1u << n) - 1u;
            }
            reinterpret_cast<uint16_t *>(pd.bits + (size_t)b * pd.bits_per_seq)[c] = (uint16_t)bits;
        }
    }
    for (int b = gwarp; b < B; b += n_gwarps) {
        const int L = padded ? extent : seq_lens[b];   // (requested with the parents: one round trip, not two)
        for (int j = lane; j < T; j += 32) par[warp][j] = parent[(size_t)b * T + j];
        __syncwarp();
        int st = warp_tree_valid(par[warp], T, lane) ? READER_OK : READER_ERR_BAD_TREE;
        if (anc_out) {
            for (int j = lane; j < T; j += 32) {
                uint64_t lo = 0, hi = 0;
                int lv = 0;
                if (st == READER_OK) node_ancestors(par[warp], T, j, lo, hi, lv);
                anc_out[((size_t)b * T + j) * 2 + 0] = lo;
                anc_out[((size_t)b * T + j) * 2 + 1] = hi;
            }
        }
        int npages = 0;
        if (padded) {
            if (!extent_ok) st = READER_ERR_CAPACITY;   // whatever the tree: no sample can be served
            else if (st == READER_OK) npages = (L + kPage - 1) / kPage;
        } else if (st == READER_OK) {
            if (L < 0 || (int64_t)L > (int64_t)max_pages * kPage) {
                st = READER_ERR_CAPACITY;
            } else {
                npages = (L + kPage - 1) / kPage;
                bool ok = true;
                for (int p = lane; p < npages; p += 32) {
                    int pg = page_table[(size_t)b * max_pages + p];
                    ok = ok && pg >= 0 && pg < num_pages;
                }
                if (!__all_sync(0xffffffffu, ok)) st = READER_ERR_BAD_PAGE;
            }
        }
        if (lane == 0) {
            status[b] = st;
            seq_ntiles[b] = st == READER_OK ? npages + n_tree_tiles : 0;
            seq_npages[b] = st == READER_OK ? npages : 0;
        }
        if (st != READER_OK && out) {   // a rejected sequence gets defined output: zero rows, zero lse
                                         // (out == nullptr: the attention calls that follow do it per layer)
            const size_t n16 = (size_t)T * Hq * D / 8;
            uint4 *o = reinterpret_cast<uint4 *>(out + (size_t)b * T * Hq * D);
            for (size_t i = lane; i < n16; i += 32) o[i] = make_uint4(0, 0, 0, 0);
            if (lse)
                for (int i = lane; i < T * Hq; i += 32) lse[(size_t)b * T * Hq + i] = 0.f;
        }
        __syncwarp();
    }
    __syncthreads();
    if (gridDim.x > 1) {
        if (threadIdx.x == 0) {
            __threadfence();   // this block's seq_ntiles before its count
            s_last = atomicAdd(error_flag + 1, 1) == (int)gridDim.x - 1;
        }
        __syncthreads();
        if (!s_last) return;
        __threadfence();
    }
    if (warp == 0) {
        int carry = 0;
        if (lane == 0) seq_tile_start[0] = 0;
        for (int base = 0; base < B; base += 32) {
            int b = base + lane;
            const int nt = b < B ? __ldcg(seq_ntiles + b) : 0;   // (possibly another block's: not through L1)
            int v = nt > 0 ? (nt + kUnitOverhead) * units_per_seq : 0;
            int incl = v;
            for (int d = 1; d < 32; d <<= 1) {
                int t = __shfl_up_sync(0xffffffffu, incl, d);
                if (lane >= d) incl += t;
            }
            if (b < B) seq_tile_start[b + 1] = carry + incl;
            carry += __shfl_sync(0xffffffffu, incl, 31);
        }
    }
}

void launch_prepare(const reader_kv_cache &c, const PaddedIn &padded, const int32_t *parent, int B, int T, int n_tree_tiles,
                    int units_per_seq, uint64_t *anc_out, int32_t *seq_tile_start, int32_t *seq_ntiles,
                    int32_t *seq_npages, int32_t *status, int32_t *error_flag, __nv_bfloat16 *out, float *lse,
                    int Hq, int D, cudaStream_t st) {
    // one block up to 64 sequences (two rounds of its 32 warps); beyond that a block per 32 sequences, up to 64 blocks
    int blocks = 1;
    if (B > 64) {
        blocks = (B + 31) / 32 < 64 ? (B + 31) / 32 : 64;
        cudaMemsetAsync(error_flag + 1, 0, sizeof(int32_t), st);   // the "blocks done" counter behind the flag
    }
    launch_pdl(prepare_kernel, dim3(blocks), dim3(1024), 0, st, padded, c.page_table, c.seq_lens, c.max_pages_per_seq, c.num_pages,
               parent, B, T, n_tree_tiles, units_per_seq, anc_out, seq_tile_start, seq_ntiles, seq_npages, status,
               error_flag, out, lse, Hq, D);
}

}  // namespace reader
