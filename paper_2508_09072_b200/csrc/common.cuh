// Shared declarations of the verification kernels: parameter blocks, the flattened
// split-KV work partition, and small device helpers.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "reader_verify.h"

namespace reader {

constexpr int kPage = READER_PAGE_SIZE;   // tokens per KV tile (= cache page)
constexpr int kTileM = 128;               // query rows per M tile
constexpr int kMaxNodes = READER_MAX_NODES;

// ---------------------------------------------------------------------------------------------
// Work partition (split-KV over a flattened tile list).
//
// A *unit* is (sequence b, KV head h, M tile mt): kTileM query rows (node j, group member g) with
// row = j * G + g, attending over ntiles(b) KV tiles: the committed pages of b followed by the
// tree tiles.  The KV streams (b, h), each kUnitOverhead overhead entries followed by its tiles in
// order, form one flat list of W entries that is cut
// into n_lanes contiguous ranges of near-equal length.  A *lane* is n_mtiles CTAs, one per M tile,
// that walk the same range: CTA c has lane c / n_mtiles and M tile c % n_mtiles.  The CTAs of a
// lane read the same K/V tiles at the same pace, so all but the first of them find the tile in
// L2 (with an independent position per M tile every one of them fetched it from HBM again).
// The part of a range that lies in one KV stream is a *segment*.  A segment that covers its whole
// unit writes the final output; any other segment writes an (m, l, O) partial into one of the
// CTA's two slots: slot 2c when the segment does not start its unit, slot 2c+1 when it does.
// ---------------------------------------------------------------------------------------------
struct Sched {
    const int32_t *seq_tile_start;  // [B+1] first flat tile of sequence b
    const int32_t *seq_ntiles;      // [B]   tiles per unit of sequence b (0: sequence skipped)
    const int32_t *seq_npages;      // [B]   committed pages among them
    int32_t n_ctas;                 // CTAs launched (n_ctas / n_mtiles lanes); effective_ctas() of the lanes share the work
    int32_t units_per_seq;          // KV streams per sequence: Hkv
    int32_t n_mtiles;               // M tiles per KV stream = CTAs per lane
    int32_t aligned;                // cut every KV stream at the same relative positions (see lane_range)
};

struct Segment {
    int b, h, mt;
    int tile_begin, tile_end;  // real tiles within the unit; may be empty (tile_end <= tile_begin)
    int span;                  // entries of the flat list this segment covers (overhead entries included)
    int unit_w0;               // flat index of the unit's first entry
    int ntiles, npages;
    int len;                   // committed length of the sequence (segment_at_warp only; 0 with a padded cache)
    bool full;                 // covers the whole unit
    int slot;                  // partial slot when !full
};

// Starting a unit costs about as much as kUnitOverhead tiles (waiting for Q, the epilogue, a partial):
// the flat list gives every unit that many extra entries at its start, so a CTA whose range holds
// more unit starts gets correspondingly fewer real tiles and all CTAs finish together.
constexpr int kUnitOverhead = 6;

constexpr int kMinTilesPerCta = 8;

// CTAs that share the W tiles of a call: all that were launched, unless that would leave fewer than
// kMinTilesPerCta tiles each (start-up, epilogue and the merge of partials cost several tiles' time,
// so a small call is better cut into few pieces).  The rest find an empty range.
__device__ __forceinline__ int effective_ctas(int n_launched, int W) {
    return max(1, min(n_launched, (W + kMinTilesPerCta - 1) / kMinTilesPerCta));
}

// floor(c * W / n) for 0 <= c <= n <= 2^15 and 0 <= W < 2^31, in 32-bit arithmetic: c W = c n (W / n) + c (W % n).
// (A 64-bit division is a few hundred dependent instructions on this GPU; the thread that located a cut
// unit's last partial with three of them held its CTA up for 2.4 us at every such segment.)
__device__ __forceinline__ int mul_div(int c, int W, int n) { return c * (W / n) + (c * (W % n)) / n; }

// First tile of CTA c's range; c >= n_ctas (a CTA left without work) gets W.
__device__ __forceinline__ int range_begin(int c, int n_ctas, int W) {
    return c >= n_ctas ? W : mul_div(c, W, n_ctas);
}

// Largest b with seq_tile_start[b] <= w (w < W).
__device__ __forceinline__ int find_seq(const int32_t *start, int B, int w) {
    int lo = 0, hi = B;  // invariant: start[lo] <= w < start[hi]
    while (hi - lo > 1) {
        int mid = (lo + hi) >> 1;
        if (start[mid] <= w) lo = mid; else hi = mid;
    }
    return lo;
}

__device__ __forceinline__ Segment segment_at(const Sched &s, int B, int cta, int w, int range_end) {
    Segment g;
    g.b = find_seq(s.seq_tile_start, B, w);
    g.ntiles = s.seq_ntiles[g.b];
    g.npages = s.seq_npages[g.b];
    const int per_unit = g.ntiles + kUnitOverhead;          // entries of one unit: overhead first, then its tiles
    int local = w - s.seq_tile_start[g.b];
    int unit = local / per_unit;
    const int pos = local - unit * per_unit;
    const int pos_end = min(per_unit, pos + (range_end - w));
    g.span = pos_end - pos;
    g.unit_w0 = w - pos;
    g.tile_begin = max(0, pos - kUnitOverhead);
    g.tile_end = max(0, pos_end - kUnitOverhead);
    g.h = unit;
    g.mt = cta % s.n_mtiles;
    g.full = (g.tile_begin == 0) && (g.tile_end == g.ntiles);
    g.slot = 2 * cta + (g.tile_begin == 0 ? 1 : 0);
    return g;
}

// The schedule of up to 32 sequences held one sequence per lane: loaded once per warp with all loads in
// flight together, so that finding a segment later costs shuffles instead of a chain of dependent global
// loads (four round trips to L2 before a CTA's first tile could be requested).  With more than 32
// sequences it stays empty and the lookups go to memory.
struct WarpSched {
    int start, ntiles, npages, len;
};
__device__ __forceinline__ WarpSched load_warp_sched(const Sched &s, const int32_t *seq_lens /*nullable*/, int B, int lane) {
    WarpSched c{0x7fffffff, 0, 0, 0};
    if (B <= 32 && lane < B) {
        c.start = s.seq_tile_start[lane];
        c.ntiles = s.seq_ntiles[lane];
        c.npages = s.seq_npages[lane];
        c.len = seq_lens ? seq_lens[lane] : 0;
    }
    return c;
}

// Same result as segment_at (plus the sequence's committed length), for a whole warp calling together.
__device__ __forceinline__ Segment segment_at_warp(const Sched &s, const WarpSched &c, const int32_t *seq_lens /*nullable*/,
                                                   int B, int cta, int w, int range_end, int lane) {
    Segment g;
    int start_b;
    if (B <= 32) {
        const unsigned le = __ballot_sync(0xffffffffu, c.start <= w);   // the starts never decrease: a prefix of the lanes
        const int b = le ? 31 - __clz(le) : 0;
        g.b = b;
        start_b = __shfl_sync(0xffffffffu, c.start, b);
        g.ntiles = __shfl_sync(0xffffffffu, c.ntiles, b);
        g.npages = __shfl_sync(0xffffffffu, c.npages, b);
        g.len = __shfl_sync(0xffffffffu, c.len, b);
    } else {
        int b = 0;
        for (int base = 0; base < B; base += 32) {   // one round of parallel loads per 32 sequences
            const int i = base + lane;
            const unsigned le = __ballot_sync(0xffffffffu, i < B && s.seq_tile_start[i] <= w);
            if (le) b = base + 31 - __clz(le);
            if (le != 0xffffffffu) break;
        }
        g.b = b;
        start_b = s.seq_tile_start[b];
        g.ntiles = s.seq_ntiles[b];
        g.npages = s.seq_npages[b];
        g.len = seq_lens ? seq_lens[b] : 0;
    }
    const int per_unit = g.ntiles + kUnitOverhead;          // entries of one unit: overhead first, then its tiles
    int local = w - start_b;
    int unit = local / per_unit;
    const int pos = local - unit * per_unit;
    const int pos_end = min(per_unit, pos + (range_end - w));
    g.span = pos_end - pos;
    g.unit_w0 = w - pos;
    g.tile_begin = max(0, pos - kUnitOverhead);
    g.tile_end = max(0, pos_end - kUnitOverhead);
    g.h = unit;
    g.mt = cta % s.n_mtiles;
    g.full = (g.tile_begin == 0) && (g.tile_end == g.ntiles);
    g.slot = 2 * cta + (g.tile_begin == 0 ? 1 : 0);
    return g;
}

// Lane (of n_ctas lanes) whose range contains flat tile w.
__device__ __forceinline__ int cta_of_tile(int w, int n_ctas, int W) {
    int c = (int)((float)w * (float)n_ctas / (float)W);   // a first guess; the loops below make it exact
    c = max(0, min(c, n_ctas - 1));
    while (c + 1 < n_ctas && range_begin(c + 1, n_ctas, W) <= w) ++c;
    while (c > 0 && range_begin(c, n_ctas, W) > w) --c;
    return c;
}

// ---------------------------------------------------------------------------------------------
// Aligned partition, for a shared prompt prefix too large to stay in L2 (Sched::aligned).
//
// With equal ranges of the flat list the lanes sit at unrelated positions of their KV streams, so the
// B sequences that share a prefix reach a given prefix tile at B different times and a prefix larger
// than L2 comes from HBM several times over (measured: 16 sequences over a 134 MB prefix read 1.08 GB).
// Here every KV stream (sequence b, KV head h) is cut at the same relative positions instead: with at
// least as many lanes as streams, stream s belongs to the k = n_lanes / n_streams lanes s*k .. s*k+k-1,
// piece j covering entries [j*len/k, (j+1)*len/k) of it; with fewer lanes, lane l walks the
// q = ceil(n_streams / n_lanes) whole streams l*q .. l*q+q-1 one after the other.  Either way all lanes
// start their piece together and advance at the same pace, so the lanes of the sequences sharing a
// prefix ask for the same prefix tile within a short time of each other: the first fetches it from HBM,
// the others find it in L2.  The price is load balance (lanes beyond n_streams * k, or the last partial
// round of streams, idle; streams of different length end at different times), which the equal-range
// partition does not pay, so it is used only where the prefix would otherwise be re-read.
// ---------------------------------------------------------------------------------------------
// First flat entry and number of entries of KV stream `stream` = b * units_per_seq + h.
__device__ __forceinline__ void stream_span(const Sched &s, int stream, int &start, int &len) {
    const int b = stream / s.units_per_seq, h = stream - b * s.units_per_seq;
    const int nt = s.seq_ntiles[b];
    len = nt > 0 ? nt + kUnitOverhead : 0;
    start = s.seq_tile_start[b] + h * len;
}

struct LaneRange {
    int w_begin, w_end;
};
// The range of the flat list that lane `lane` of n_lanes walks; a lane without work gets an empty range.
__device__ __forceinline__ LaneRange lane_range(const Sched &s, int B, int lane, int n_lanes, int W) {
    if (!s.aligned) return LaneRange{range_begin(lane, n_lanes, W), range_begin(lane + 1, n_lanes, W)};
    const int n_streams = B * s.units_per_seq;
    if (lane >= n_lanes) return LaneRange{W, W};
    int start, len;
    if (n_lanes >= n_streams) {
        const int k = n_lanes / n_streams;
        const int st = lane / k, j = lane - st * k;
        if (st >= n_streams) return LaneRange{W, W};
        stream_span(s, st, start, len);
        return LaneRange{start + mul_div(j, len, k), start + mul_div(j + 1, len, k)};
    }
    const int q = (n_streams + n_lanes - 1) / n_lanes;
    const int s0 = lane * q, s1 = min(n_streams, s0 + q);
    if (s0 >= n_streams) return LaneRange{W, W};
    stream_span(s, s0, start, len);
    int last_start, last_len;
    stream_span(s, s1 - 1, last_start, last_len);
    return LaneRange{start, last_start + last_len};
}

// Lane whose range contains flat entry w, which lies in the unit of segment g (any segment of that unit).
__device__ __forceinline__ int lane_of_entry(const Sched &s, int B, const Segment &g, int w, int n_lanes, int W) {
    if (!s.aligned) return cta_of_tile(w, n_lanes, W);
    const int n_streams = B * s.units_per_seq;
    const int st = g.b * s.units_per_seq + g.h;
    if (n_lanes >= n_streams) {
        const int k = n_lanes / n_streams;
        const int len = g.ntiles + kUnitOverhead, pos = w - g.unit_w0;
        int j = (int)((float)pos * (float)k / (float)len);   // a first guess, made exact below
        j = max(0, min(j, k - 1));
        while (j + 1 < k && mul_div(j + 1, len, k) <= pos) ++j;
        while (j > 0 && mul_div(j, len, k) > pos) --j;
        return st * k + j;
    }
    return st / ((n_streams + n_lanes - 1) / n_lanes);
}

// The work of one CTA: its M tile and its lane's range of the flat tile list.
struct CtaWork {
    int mt, n_lanes, w_begin, w_end;
};
__device__ __forceinline__ CtaWork cta_work(const Sched &s, int B, int cta, int W) {
    CtaWork k;
    const int lane = cta / s.n_mtiles;
    k.mt = cta - lane * s.n_mtiles;
    k.n_lanes = effective_ctas(s.n_ctas / s.n_mtiles, W);   // lanes that share the work
    const LaneRange r = lane_range(s, B, lane, k.n_lanes, W);   // a lane left without work gets an empty range
    k.w_begin = r.w_begin;
    k.w_end = r.w_end;
    return k;
}

// Written by the attention CTA that starts a unit it does not finish (at most one per CTA); read by
// the combine kernel.  b < 0: this CTA started no such unit.
struct SplitDesc {
    int32_t b, h, mt, c_last;   // unit, and the last CTA holding one of its partials
};

// Called by one thread per segment: if the segment starts its unit without finishing it, note where
// the unit's partials end so that the combine kernel can find them without any search.
__device__ __forceinline__ void record_split(SplitDesc *desc, const Sched &s, int B, int n_lanes, const Segment &g, int cta, int W) {
    if (g.tile_begin != 0 || g.full || g.tile_end <= g.tile_begin) return;
    SplitDesc d;
    d.b = g.b; d.h = g.h; d.mt = g.mt;
    d.c_last = lane_of_entry(s, B, g, g.unit_w0 + kUnitOverhead + g.ntiles - 1, n_lanes, W) * s.n_mtiles + g.mt;   // same M tile, last lane
    desc[cta] = d;
}

// ---------------------------------------------------------------------------------------------
// Attention parameters
// ---------------------------------------------------------------------------------------------
struct AttnParams {
    const __nv_bfloat16 *q, *k_tree, *v_tree, *k_pool, *v_pool;
    const int32_t *page_table;
    const int32_t *seq_lens;
    const uint64_t *anc;       // [B][T][2]
    __nv_bfloat16 *out;
    float *lse;                // nullable
    float *partial_o;          // [slots][kTileM][D]
    float *partial_ml;         // [slots][kTileM][2]  (m in log2 units, l)
    SplitDesc *split_desc;     // [n_ctas]
    int32_t *status;           // [B]
    int32_t *error_flag;       // one word in the workspace: set on a bounded-wait timeout
    int B, T, Hq, Hkv, D, G;
    int max_pages, num_pages;
    int64_t pool_rows;         // rows of head_dim elements in k_pool / v_pool (what a TMA descriptor may cover)
    int shared_prefix_pages;   // leading page-table entries common to every sequence
    float scale_log2;          // softmax_scale * log2(e)
    // Padded batch cache (Sec. 4.3) instead of the paged one when valid_bits != nullptr: k_pool / v_pool
    // are then [B][Hkv][cap][D], tile t of (b, h) starts at row (b * Hkv + h) * cap + t * kPage, there is
    // no page table and no per-sequence length, and bit r of valid_bits[b * bits_per_seq + t] tells
    // whether row t * kPage + r of sample b is a real entry (0 at and beyond the common extent).
    const uint64_t *valid_bits;
    int bits_per_seq, cap;
    int zero_rejected;         // the combine kernel zeroes the rows of sequences whose status word is set (the
                               // preparation ran in an earlier call and could not know this call's output)
    const int32_t *parent;     // [B][T] (the single-launch kernel for small calls checks the trees itself)
    Sched sched;
};

// Committed length of sequence b (unused, 0, with the padded cache: its tiles carry their own masks).
__device__ __forceinline__ int committed_len(const AttnParams &p, int b) { return p.valid_bits ? 0 : p.seq_lens[b]; }

// Keys of committed tile t of sequence b that its queries may see, bit r = key t * kPage + r.
__device__ __forceinline__ uint64_t page_visible(const AttnParams &p, int b, int t, int L) {
    if (p.valid_bits) return p.valid_bits[(size_t)b * p.bits_per_seq + t];
    const int valid = L - t * kPage;
    return valid >= kPage ? ~0ull : ((1ull << valid) - 1);
}

// First row of committed tile t of KV stream (b, h) in the [rows][D] view of a pool.
__device__ __forceinline__ int64_t page_first_row(const AttnParams &p, int b, int h, int t, int page) {
    if (p.valid_bits) return ((int64_t)b * p.Hkv + h) * p.cap + (int64_t)t * kPage;
    return ((int64_t)page * p.Hkv + h) * kPage;
}

__device__ __forceinline__ float bf16lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16hi(uint32_t u) { return __uint_as_float(u & 0xffff0000u); }

// Launch with programmatic stream serialization: the kernel may be scheduled while its predecessor
// in the stream is still running.  Every kernel launched this way starts with pdl_wait(), which
// blocks until that predecessor has completed and its writes are visible; only launch latency is
// hidden, never a data dependency.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args &&...args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Column ranges a logits row is cut into by the argmax scan (reader_accept, reader_accept_commit,
// reader_accept_noalloc): enough blocks to fill the GPU when rows are few, at least three per row (one
// 513 KB block per row left the scan short of bytes in flight), at least 2048 columns each, at most
// kMaxArgmaxSplits (what the partial arrays are sized for).
constexpr int kMaxArgmaxSplits = 64;
inline int argmax_splits(int n_sm, int64_t rows, int64_t vocab) {
    int64_t want = (4 * (int64_t)n_sm + rows - 1) / rows;
    if (want < 3) want = 3;
    const int64_t cap = vocab / 2048 > 0 ? vocab / 2048 : 1;
    if (want > cap) want = cap;
    if (want > kMaxArgmaxSplits) want = kMaxArgmaxSplits;
    return (int)want;
}

// Host-side launchers (one per .cu file)
void launch_tree_encode(const int32_t *parent, int B, int T, uint64_t *anc, int32_t *level,
                        int32_t *status, cudaStream_t st);
// The padded batch cache as the preparation kernel sees it (valid == nullptr: the paged cache is used).
struct PaddedIn {
    const uint8_t *valid;     // [B][cap]
    const int32_t *extent;    // device scalar: the common length
    int cap;
    uint64_t *bits;           // out: [B][bits_per_seq], the mask packed per tile, cleared from the extent on
    int bits_per_seq;
};
void launch_prepare(const reader_kv_cache &c, const PaddedIn &padded, const int32_t *parent, int B, int T, int n_tree_tiles,
                    int units_per_seq, uint64_t *anc_out /*nullable*/, int32_t *seq_tile_start,
                    int32_t *seq_ntiles, int32_t *seq_npages, int32_t *status, int32_t *error_flag,
                    __nv_bfloat16 *out, float *lse /*nullable*/, int Hq, int D, cudaStream_t st);
void launch_padded_append(__nv_bfloat16 *k, __nv_bfloat16 *v, int B, int Hkv, int cap, int D, uint8_t *valid,
                          int32_t *extent, const __nv_bfloat16 *k_tree, const __nv_bfloat16 *v_tree, int T,
                          const int32_t *path, const int32_t *n_acc, int max_path, int32_t *status, cudaStream_t st);
void launch_set_extent(const int32_t *lengths, int B, int32_t *extent, cudaStream_t st);
void launch_attn_generic(const AttnParams &p, cudaStream_t st);
void launch_combine(const AttnParams &p, cudaStream_t st);
void launch_argmax(const float *logits, int64_t rows, int64_t vocab, int splits, float *part_val,
                   int32_t *part_idx, cudaStream_t st);
void launch_sample(const float *logits, int64_t rows, int64_t vocab, const int32_t *parent, const float *uniforms,
                   int T, float c, int64_t top_k, float top_p, int32_t *target, int n_sm, cudaStream_t st);
int sample_max_vocab();
void launch_kv_rearrange(__nv_bfloat16 *k, __nv_bfloat16 *v, int B, int Hkv, int cap, int D, uint8_t *valid,
                         int32_t *lengths, cudaStream_t st);
void launch_accept(const int32_t *parent, const int32_t *tok, int32_t *target, int B, int T,
                   int max_path, const float *part_val, const int32_t *part_idx, int splits,
                   int32_t *path, int32_t *n_acc, int32_t *bonus, int32_t *status, cudaStream_t st);
void launch_accept_commit(const int32_t *parent, const int32_t *tok, int32_t *target, int B, int T, int max_path,
                          const float *part_val, const int32_t *part_idx, int splits, int32_t *path, int32_t *n_acc,
                          int32_t *bonus, int32_t *status, const reader_kv_cache &c, const __nv_bfloat16 *k_tree,
                          const __nv_bfloat16 *v_tree, int update_seq_lens, int32_t *slots, int32_t *commit_status,
                          cudaStream_t st);
// Pool and tree pointers of up to kCommitLayersPerLaunch layers, passed to the kernel by value.
constexpr int kCommitLayersPerLaunch = 32;
struct CommitLayers {
    __nv_bfloat16 *k_pool[kCommitLayersPerLaunch], *v_pool[kCommitLayersPerLaunch];
    const __nv_bfloat16 *k_tree[kCommitLayersPerLaunch], *v_tree[kCommitLayersPerLaunch];
};
void launch_kv_commit_layers(const reader_kv_cache &c, const CommitLayers *chunks, int n_layers, int B, int T,
                             const int32_t *path, const int32_t *n_acc, int max_path, int update_seq_lens,
                             int32_t *slots, int32_t *status, cudaStream_t st);
void launch_kv_commit(const reader_kv_cache &c, const __nv_bfloat16 *k_tree, const __nv_bfloat16 *v_tree,
                      int B, int T, const int32_t *path, const int32_t *n_acc, int max_path,
                      int update_seq_lens, int32_t *slots, int32_t *status, cudaStream_t st);

}  // namespace reader
