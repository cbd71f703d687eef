// C-ABI entry points: argument validation, workspace carving and kernel sequencing.
// Nothing here touches device data from the host or synchronises the stream.
#include <new>
#include <vector>

#include "common.cuh"
#include "ctx.cuh"


namespace {

using namespace reader;

constexpr int kMaxSplits = kMaxArgmaxSplits;
constexpr int kSmallTilesPerCta = 24;   // largest share of a unit that still counts as a small call (measured: the
                                        // single launch wins by 18-24 % at 15-16 tiles per CTA and ties at 29-32)
constexpr int64_t kAlignedPrefixBytes = 48ll << 20;   // shared prefix K+V above which the lanes walk it in step (L2: 126 MB)
constexpr size_t kAlign = 256;

inline size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }
inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

struct WsLayout {
    size_t error_flag, seq_tile_start, seq_ntiles, seq_npages, anc, split_desc, partial_ml, partial_o, amax_val, amax_idx, total;
};

inline int max_ctas(const reader_ctx *ctx) { return 2 * ctx->n_sm; }

WsLayout ws_layout(const reader_ctx *ctx, int B, int T, int D) {
    WsLayout w{};
    size_t at = 0;
    auto take = [&](size_t bytes) { size_t o = at; at = align_up(at + bytes); return o; };
    const size_t slots = 2 * (size_t)max_ctas(ctx);
    w.error_flag = take(2 * sizeof(int32_t));   // the flag; behind it the preparation kernel's "blocks done" counter
    w.seq_tile_start = take(sizeof(int32_t) * ((size_t)B + 1));
    w.seq_ntiles = take(sizeof(int32_t) * (size_t)B);
    w.seq_npages = take(sizeof(int32_t) * (size_t)B);
    w.anc = take(sizeof(uint64_t) * 2 * (size_t)B * T);
    w.split_desc = take(sizeof(SplitDesc) * (size_t)max_ctas(ctx));
    w.partial_ml = take(sizeof(float) * 2 * slots * kTileM);
    w.partial_o = take(sizeof(float) * slots * kTileM * (size_t)D);
    w.amax_val = take(sizeof(float) * (size_t)B * T * kMaxSplits);
    w.amax_idx = take(sizeof(int32_t) * (size_t)B * T * kMaxSplits);
    w.total = at;
    return w;
}

inline bool shape_ok(int B, int T, int Hq, int Hkv, int D) {
    return B >= 0 && T >= 1 && T <= kMaxNodes && Hq >= 1 && Hkv >= 1 && Hq % Hkv == 0 && (D == 64 || D == 128);
}

inline reader_status check_device(const reader_ctx *ctx) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return READER_ERR_CUDA;
    return dev == ctx->device ? READER_OK : READER_ERR_INVALID_ARG;
}

inline reader_status launch_status() { return cudaGetLastError() == cudaSuccess ? READER_OK : READER_ERR_CUDA; }

}  // namespace

extern "C" {

reader_status reader_create(reader_ctx **out, int device) {
    if (!out) return READER_ERR_INVALID_ARG;
    *out = nullptr;
    int n_sm = 0, major = 0;
    if (cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, device) != cudaSuccess ||
        cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device) != cudaSuccess) {
        cudaGetLastError();
        return READER_ERR_CUDA;
    }
    if (major != 10) return READER_ERR_UNSUPPORTED;   // the kernels are sm_100a code only
    reader_ctx *ctx = new (std::nothrow) reader_ctx();
    if (!ctx) return READER_ERR_CUDA;
    ctx->device = device;
    ctx->n_sm = n_sm;
    ctx->attn_kernel = 0;
    ctx->partition = 0;
    ctx->ev_start = ctx->ev_stop = nullptr;
    ctx->ev_acc_start = ctx->ev_acc_stop = nullptr;
    ctx->prepared = PreparedRecord{};
    reader_status st = sm100_host_init(&ctx->sm100, device);
    if (st != READER_OK) {
        delete ctx;
        return st;
    }
    *out = ctx;
    return READER_OK;
}

void reader_destroy(reader_ctx *ctx) {
    if (!ctx) return;
    sm100_host_destroy(&ctx->sm100);
    delete ctx;
}

const char *reader_status_string(reader_status s) {
    switch (s) {
        case READER_OK: return "ok";
        case READER_ERR_INVALID_ARG: return "invalid argument";
        case READER_ERR_BAD_TREE: return "parent array is not a tree rooted at node 0 with parent[j] < j";
        case READER_ERR_CAPACITY: return "page table cannot hold the requested positions";
        case READER_ERR_WORKSPACE: return "workspace too small";
        case READER_ERR_UNSUPPORTED: return "unsupported shape or device";
        case READER_ERR_TIMEOUT: return "a bounded device-side wait gave up";
        case READER_ERR_CUDA: return "CUDA call failed";
        case READER_ERR_BAD_PAGE: return "page id outside the pool";
        case READER_ERR_TOO_LARGE: return "problem larger than the built-in scratch of the allocation-free entry point";
    }
    return "unknown status";
}

reader_status reader_set_attn_kernel(reader_ctx *ctx, int32_t which) {
    if (!ctx || which < 0 || which > 3) return READER_ERR_INVALID_ARG;
    ctx->attn_kernel = which;
    return READER_OK;
}

reader_status reader_set_partition(reader_ctx *ctx, int32_t which) {
    if (!ctx || which < 0 || which > 2) return READER_ERR_INVALID_ARG;
    ctx->partition = which;
    return READER_OK;
}

reader_status reader_set_timing_events(reader_ctx *ctx, void *start, void *stop) {
    if (!ctx || ((start == nullptr) != (stop == nullptr))) return READER_ERR_INVALID_ARG;
    ctx->ev_start = (cudaEvent_t)start;
    ctx->ev_stop = (cudaEvent_t)stop;
    return READER_OK;
}

reader_status reader_set_accept_timing_events(reader_ctx *ctx, void *start, void *stop) {
    if (!ctx || ((start == nullptr) != (stop == nullptr))) return READER_ERR_INVALID_ARG;
    ctx->ev_acc_start = (cudaEvent_t)start;
    ctx->ev_acc_stop = (cudaEvent_t)stop;
    return READER_OK;
}

size_t reader_workspace_bytes(const reader_ctx *ctx, int32_t max_batch, int32_t max_nodes, int32_t n_q_heads,
                              int32_t n_kv_heads, int32_t head_dim) {
    if (!ctx || !shape_ok(max_batch, max_nodes, n_q_heads, n_kv_heads, head_dim)) return 0;
    return ws_layout(ctx, max_batch, max_nodes, head_dim).total;
}

reader_status reader_tree_encode(reader_ctx *ctx, const int32_t *parent, int32_t batch, int32_t n_nodes,
                                 uint64_t *anc_mask_out, int32_t *level_out, int32_t *status_out, void *stream) {
    if (!ctx || !parent || !anc_mask_out || !status_out || batch < 0 || n_nodes < 1 || n_nodes > kMaxNodes ||
        !aligned16(anc_mask_out))
        return READER_ERR_INVALID_ARG;
    if (reader_status st = check_device(ctx)) return st;
    launch_tree_encode(parent, batch, n_nodes, anc_mask_out, level_out, status_out, (cudaStream_t)stream);
    return launch_status();
}

}  // extern "C"

namespace {

// What the two attention entry points share once their cache-specific arguments are checked: the
// workspace is carved, the parameter block completed and the three kernels are enqueued.
// `p` arrives with the cache fields set; `bits_offset` is where the packed mask of a padded cache
// lives in the workspace (unused for the paged cache).
enum AttnMode { kPrepareAndRun, kPrepareOnly, kRunPrepared };

reader_status run_verify_attn(reader_ctx *ctx, AttnParams p, const reader_kv_cache *paged, const reader_padded_cache *padded,
                              const reader_tree *tree, float softmax_scale, void *workspace, size_t workspace_bytes,
                              void *stream, AttnMode mode = kPrepareAndRun) {
    const int B = p.B, T = p.T, Hkv = p.Hkv, D = p.D;
    const int n_mtiles = (T * p.G + kTileM - 1) / kTileM;
    const int n_tree_tiles = (T + kPage - 1) / kPage;
    const int64_t max_pages = padded ? ((int64_t)padded->capacity + kPage - 1) / kPage : paged->max_pages_per_seq;
    const int64_t tiles_bound = (int64_t)B * Hkv * n_mtiles * (max_pages + n_tree_tiles + kUnitOverhead);
    if (tiles_bound >= (int64_t)1 << 31) return READER_ERR_UNSUPPORTED;
    if (n_mtiles > max_ctas(ctx)) return READER_ERR_UNSUPPORTED;   // a lane holds one CTA per M tile of a KV stream
    const WsLayout w = ws_layout(ctx, B, T, D);
    const size_t bits_bytes = padded ? align_up(sizeof(uint64_t) * (size_t)B * (size_t)max_pages) : 0;
    if (workspace_bytes < w.total + bits_bytes) return READER_ERR_WORKSPACE;
    if (reader_status st = check_device(ctx)) return st;

    unsigned char *ws = static_cast<unsigned char *>(workspace);
    cudaStream_t st = (cudaStream_t)stream;
    p.anc = tree->anc_mask ? tree->anc_mask : reinterpret_cast<const uint64_t *>(ws + w.anc);
    p.partial_o = reinterpret_cast<float *>(ws + w.partial_o);
    p.partial_ml = reinterpret_cast<float *>(ws + w.partial_ml);
    p.split_desc = reinterpret_cast<SplitDesc *>(ws + w.split_desc);
    p.error_flag = reinterpret_cast<int32_t *>(ws + w.error_flag);
    p.scale_log2 = softmax_scale * 1.4426950408889634f;
    p.sched.seq_tile_start = reinterpret_cast<const int32_t *>(ws + w.seq_tile_start);
    p.sched.seq_ntiles = reinterpret_cast<const int32_t *>(ws + w.seq_ntiles);
    p.sched.seq_npages = reinterpret_cast<const int32_t *>(ws + w.seq_npages);
    p.sched.units_per_seq = Hkv;
    p.sched.n_mtiles = n_mtiles;
    // A shared prefix whose K and V exceed a good part of the L2 is walked by all sequences' lanes in step
    // (the aligned partition of common.cuh), so that it comes from HBM once; a smaller one stays in L2
    // whatever the order, and the equal-range partition balances ragged suffixes better.
    p.sched.aligned = (paged && B >= 2 && (int64_t)p.shared_prefix_pages * Hkv * kPage * D * 2 * 2 > kAlignedPrefixBytes) ? 1 : 0;
    if (ctx->partition == 1) p.sched.aligned = 0;
    if (ctx->partition == 2) p.sched.aligned = (paged && B >= 2 && p.shared_prefix_pages > 0) ? 1 : 0;
    PaddedIn pin{};
    reader_kv_cache none{};
    if (padded) {
        pin.valid = padded->valid;
        pin.extent = padded->extent;
        pin.cap = padded->capacity;
        pin.bits = reinterpret_cast<uint64_t *>(ws + w.total);
        pin.bits_per_seq = (int)max_pages;
        p.valid_bits = pin.bits;
        p.bits_per_seq = pin.bits_per_seq;
        p.cap = padded->capacity;
    }

    const bool tc_ok = sm100_supports(&ctx->sm100, p, softmax_scale);
    if (ctx->attn_kernel >= 2 && !tc_ok && mode != kPrepareOnly) return READER_ERR_UNSUPPORTED;
    const bool use_tc = tc_ok && ctx->attn_kernel != 1;
    // A call with few units (one or a few sequences: the batch-1 regime of Sec. 4.1) is three dependent
    // launches of mostly latency on the general path.  It takes one launch instead: every unit
    // (sequence, KV head, M tile) gets a cluster of up to 8 CTAs that checks the sequence, shares the unit's
    // tiles and merges the shares in distributed shared memory.  Chosen when the clusters fit the GPU in one
    // wave and a share is at most kSmallTilesPerCta tiles (going by the page table's width: lengths live on
    // the device); reader_set_attn_kernel(3) takes it whenever the clusters fit.
    int small_cluster = 0;
    p.parent = tree->parent;
    if (use_tc && paged && !p.sched.aligned && ctx->attn_kernel != 2) {
        const int64_t n_units = (int64_t)B * Hkv * n_mtiles, bound = max_pages + n_tree_tiles;
        int cs = 8;
        while (cs > 1 && (bound < 2 * cs || n_units * cs > max_ctas(ctx))) cs >>= 1;
        const bool fits = n_units * cs <= max_ctas(ctx);
        if (fits && (ctx->attn_kernel == 3 || (bound + cs - 1) / cs <= kSmallTilesPerCta)) small_cluster = cs;
    }
    if (ctx->attn_kernel == 3 && small_cluster == 0 && mode != kPrepareOnly) return READER_ERR_UNSUPPORTED;
    if (small_cluster > 0 && mode == kPrepareAndRun && !tree->anc_mask) p.anc = nullptr;   // no preparation runs: masks from the parent array
    // Two resident CTAs per SM for both kernels -- fewer when the page table is too narrow to give that many
    // CTAs work: on the device effective_ctas() never uses more than ceil(W / kMinTilesPerCta) lanes, and W
    // cannot exceed the bound below, so the partition is the same and the launches are smaller.
    {
        const int64_t w_bound = (int64_t)B * Hkv * (max_pages + n_tree_tiles + kUnitOverhead);
        const int64_t lanes = (w_bound + kMinTilesPerCta - 1) / kMinTilesPerCta;
        const int64_t busy = (lanes < 1 ? 1 : lanes) * n_mtiles;
        p.sched.n_ctas = (int)(busy < max_ctas(ctx) ? busy : max_ctas(ctx));
    }

    if (mode == kPrepareOnly || (mode == kPrepareAndRun && small_cluster == 0))
        launch_prepare(paged ? *paged : none, pin, tree->parent, B, T, n_tree_tiles, p.sched.units_per_seq,
                   tree->anc_mask ? nullptr : reinterpret_cast<uint64_t *>(ws + w.anc),
                   reinterpret_cast<int32_t *>(ws + w.seq_tile_start), reinterpret_cast<int32_t *>(ws + w.seq_ntiles),
                   reinterpret_cast<int32_t *>(ws + w.seq_npages), p.status, p.error_flag, p.out, p.lse, p.Hq, D, st);
    if (mode == kPrepareOnly) return launch_status();
    if (ctx->ev_start) cudaEventRecord(ctx->ev_start, st);
    if (use_tc) {
        if (reader_status s = launch_attn_sm100(&ctx->sm100, p, small_cluster, st)) return s;
    } else {
        launch_attn_generic(p, st);
    }
    if (ctx->ev_stop) cudaEventRecord(ctx->ev_stop, st);
    if (small_cluster == 0) launch_combine(p, st);
    return launch_status();
}

}  // namespace

extern "C" {

reader_status reader_verify_attn(reader_ctx *ctx, const void *q, int32_t n_q_heads, const void *k_tree,
                                 const void *v_tree, const reader_kv_cache *cache, const reader_tree *tree,
                                 float softmax_scale, void *out, float *lse_out, void *workspace,
                                 size_t workspace_bytes, int32_t *status_out, void *stream) {
    if (!ctx || !cache || !tree) return READER_ERR_INVALID_ARG;
    if (tree->batch == 0) return READER_OK;   // an empty batch has no tensors to point at
    if (!q || !k_tree || !v_tree || !out || !workspace || !status_out) return READER_ERR_INVALID_ARG;
    const int B = tree->batch, T = tree->n_nodes, Hq = n_q_heads, Hkv = cache->n_kv_heads, D = cache->head_dim;
    if (!cache->k_pool || !cache->v_pool || !cache->page_table || !cache->seq_lens || !tree->parent)
        return READER_ERR_INVALID_ARG;
    if (B < 0 || T < 1 || T > kMaxNodes || Hq < 1 || Hkv < 1 || cache->num_pages < 0 ||
        cache->max_pages_per_seq < 1 || !(softmax_scale == softmax_scale))
        return READER_ERR_INVALID_ARG;
    if (Hq % Hkv != 0 || (D != 64 && D != 128) || cache->page_size != kPage) return READER_ERR_UNSUPPORTED;
    if (cache->shared_prefix_len < 0 || cache->shared_prefix_len % kPage != 0) return READER_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k_tree) || !aligned16(v_tree) || !aligned16(cache->k_pool) ||
        !aligned16(cache->v_pool) || !aligned16(out) || !aligned16(tree->anc_mask) ||
        (reinterpret_cast<uintptr_t>(workspace) % kAlign) != 0)
        return READER_ERR_INVALID_ARG;
    AttnParams p{};
    p.q = static_cast<const __nv_bfloat16 *>(q);
    p.k_tree = static_cast<const __nv_bfloat16 *>(k_tree);
    p.v_tree = static_cast<const __nv_bfloat16 *>(v_tree);
    p.k_pool = static_cast<const __nv_bfloat16 *>(cache->k_pool);
    p.v_pool = static_cast<const __nv_bfloat16 *>(cache->v_pool);
    p.page_table = cache->page_table;
    p.seq_lens = cache->seq_lens;
    p.out = static_cast<__nv_bfloat16 *>(out);
    p.lse = lse_out;
    p.status = status_out;
    p.B = B; p.T = T; p.Hq = Hq; p.Hkv = Hkv; p.D = D; p.G = Hq / Hkv;
    p.max_pages = cache->max_pages_per_seq;
    p.num_pages = cache->num_pages;
    p.pool_rows = (int64_t)cache->num_pages * Hkv * kPage;
    p.shared_prefix_pages = cache->shared_prefix_len / kPage;
    return run_verify_attn(ctx, p, cache, nullptr, tree, softmax_scale, workspace, workspace_bytes, stream);
}

reader_status reader_verify_prepare(reader_ctx *ctx, const reader_kv_cache *cache, const reader_tree *tree,
                                    int32_t n_q_heads, void *workspace, size_t workspace_bytes, int32_t *status_out,
                                    void *stream) {
    if (!ctx || !cache || !tree) return READER_ERR_INVALID_ARG;
    ctx->prepared.valid = false;
    if (tree->batch == 0) return READER_OK;
    if (!workspace || !status_out || !cache->page_table || !cache->seq_lens || !tree->parent) return READER_ERR_INVALID_ARG;
    const int B = tree->batch, T = tree->n_nodes, Hq = n_q_heads, Hkv = cache->n_kv_heads, D = cache->head_dim;
    if (B < 0 || T < 1 || T > kMaxNodes || Hq < 1 || Hkv < 1 || cache->num_pages < 0 || cache->max_pages_per_seq < 1)
        return READER_ERR_INVALID_ARG;
    if (Hq % Hkv != 0 || (D != 64 && D != 128) || cache->page_size != kPage) return READER_ERR_UNSUPPORTED;
    if (cache->shared_prefix_len < 0 || cache->shared_prefix_len % kPage != 0) return READER_ERR_INVALID_ARG;
    if (!aligned16(tree->anc_mask) || (reinterpret_cast<uintptr_t>(workspace) % kAlign) != 0) return READER_ERR_INVALID_ARG;
    AttnParams p{};
    p.page_table = cache->page_table;
    p.seq_lens = cache->seq_lens;
    p.status = status_out;
    p.B = B; p.T = T; p.Hq = Hq; p.Hkv = Hkv; p.D = D; p.G = Hq / Hkv;
    p.max_pages = cache->max_pages_per_seq;
    p.num_pages = cache->num_pages;
    p.pool_rows = (int64_t)cache->num_pages * Hkv * kPage;
    p.shared_prefix_pages = cache->shared_prefix_len / kPage;
    const reader_status s = run_verify_attn(ctx, p, cache, nullptr, tree, 1.0f, workspace, workspace_bytes, stream, kPrepareOnly);
    if (s != READER_OK) return s;
    PreparedRecord &r = ctx->prepared;
    r.valid = true;
    r.workspace = workspace; r.page_table = cache->page_table; r.seq_lens = cache->seq_lens;
    r.parent = tree->parent; r.anc_mask = tree->anc_mask; r.status = status_out;
    r.B = B; r.T = T; r.Hq = Hq; r.Hkv = Hkv; r.D = D;
    r.max_pages = cache->max_pages_per_seq; r.num_pages = cache->num_pages; r.shared_prefix_len = cache->shared_prefix_len;
    return READER_OK;
}

reader_status reader_verify_attn_prepared(reader_ctx *ctx, const void *q, int32_t n_q_heads, const void *k_tree,
                                          const void *v_tree, const reader_kv_cache *cache, const reader_tree *tree,
                                          float softmax_scale, void *out, float *lse_out, void *workspace,
                                          size_t workspace_bytes, void *stream) {
    if (!ctx || !cache || !tree) return READER_ERR_INVALID_ARG;
    if (tree->batch == 0) return READER_OK;
    if (!q || !k_tree || !v_tree || !out || !workspace || !cache->k_pool || !cache->v_pool) return READER_ERR_INVALID_ARG;
    const PreparedRecord &r = ctx->prepared;
    const int B = tree->batch, T = tree->n_nodes, Hq = n_q_heads, Hkv = cache->n_kv_heads, D = cache->head_dim;
    // the schedule in the workspace was made for one problem: same workspace, batch, tree and block table only
    if (!r.valid || r.workspace != workspace || r.B != B || r.T != T || r.Hq != Hq || r.Hkv != Hkv || r.D != D ||
        r.page_table != cache->page_table || r.seq_lens != cache->seq_lens || r.max_pages != cache->max_pages_per_seq ||
        r.num_pages != cache->num_pages || r.shared_prefix_len != cache->shared_prefix_len || r.parent != tree->parent ||
        r.anc_mask != tree->anc_mask || cache->page_size != kPage || !(softmax_scale == softmax_scale))
        return READER_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k_tree) || !aligned16(v_tree) || !aligned16(cache->k_pool) || !aligned16(cache->v_pool) ||
        !aligned16(out))
        return READER_ERR_INVALID_ARG;
    AttnParams p{};
    p.q = static_cast<const __nv_bfloat16 *>(q);
    p.k_tree = static_cast<const __nv_bfloat16 *>(k_tree);
    p.v_tree = static_cast<const __nv_bfloat16 *>(v_tree);
    p.k_pool = static_cast<const __nv_bfloat16 *>(cache->k_pool);
    p.v_pool = static_cast<const __nv_bfloat16 *>(cache->v_pool);
    p.page_table = cache->page_table;
    p.seq_lens = cache->seq_lens;
    p.out = static_cast<__nv_bfloat16 *>(out);
    p.lse = lse_out;
    p.status = r.status;
    p.zero_rejected = 1;
    p.B = B; p.T = T; p.Hq = Hq; p.Hkv = Hkv; p.D = D; p.G = Hq / Hkv;
    p.max_pages = cache->max_pages_per_seq;
    p.num_pages = cache->num_pages;
    p.pool_rows = (int64_t)cache->num_pages * Hkv * kPage;
    p.shared_prefix_pages = cache->shared_prefix_len / kPage;
    return run_verify_attn(ctx, p, cache, nullptr, tree, softmax_scale, workspace, workspace_bytes, stream, kRunPrepared);
}

size_t reader_padded_workspace_bytes(const reader_ctx *ctx, int32_t max_batch, int32_t max_nodes, int32_t n_q_heads,
                                     int32_t n_kv_heads, int32_t head_dim, int32_t capacity) {
    if (!ctx || capacity < 1 || !shape_ok(max_batch, max_nodes, n_q_heads, n_kv_heads, head_dim)) return 0;
    const size_t words = (size_t)max_batch * (((size_t)capacity + kPage - 1) / kPage);
    return ws_layout(ctx, max_batch, max_nodes, head_dim).total + align_up(sizeof(uint64_t) * words);
}

reader_status reader_verify_attn_padded(reader_ctx *ctx, const void *q, int32_t n_q_heads, const void *k_tree,
                                        const void *v_tree, const reader_padded_cache *cache, const reader_tree *tree,
                                        float softmax_scale, void *out, float *lse_out, void *workspace,
                                        size_t workspace_bytes, int32_t *status_out, void *stream) {
    if (!ctx || !cache || !tree) return READER_ERR_INVALID_ARG;
    if (tree->batch == 0) return READER_OK;
    if (!q || !k_tree || !v_tree || !out || !workspace || !status_out) return READER_ERR_INVALID_ARG;
    const int B = tree->batch, T = tree->n_nodes, Hq = n_q_heads, Hkv = cache->n_kv_heads, D = cache->head_dim;
    if (!cache->k || !cache->v || !cache->valid || !cache->extent || !tree->parent) return READER_ERR_INVALID_ARG;
    if (B < 0 || T < 1 || T > kMaxNodes || Hq < 1 || Hkv < 1 || cache->capacity < 1 || !(softmax_scale == softmax_scale))
        return READER_ERR_INVALID_ARG;
    if (Hq % Hkv != 0 || (D != 64 && D != 128)) return READER_ERR_UNSUPPORTED;
    if (!aligned16(q) || !aligned16(k_tree) || !aligned16(v_tree) || !aligned16(cache->k) || !aligned16(cache->v) ||
        !aligned16(out) || !aligned16(tree->anc_mask) || (reinterpret_cast<uintptr_t>(workspace) % kAlign) != 0)
        return READER_ERR_INVALID_ARG;
    AttnParams p{};
    p.q = static_cast<const __nv_bfloat16 *>(q);
    p.k_tree = static_cast<const __nv_bfloat16 *>(k_tree);
    p.v_tree = static_cast<const __nv_bfloat16 *>(v_tree);
    p.k_pool = static_cast<const __nv_bfloat16 *>(cache->k);
    p.v_pool = static_cast<const __nv_bfloat16 *>(cache->v);
    p.out = static_cast<__nv_bfloat16 *>(out);
    p.lse = lse_out;
    p.status = status_out;
    p.B = B; p.T = T; p.Hq = Hq; p.Hkv = Hkv; p.D = D; p.G = Hq / Hkv;
    p.pool_rows = (int64_t)B * Hkv * cache->capacity;
    return run_verify_attn(ctx, p, nullptr, cache, tree, softmax_scale, workspace, workspace_bytes, stream);
}

reader_status reader_padded_append(reader_ctx *ctx, reader_padded_cache *cache, const void *k_tree, const void *v_tree,
                                   int32_t batch, int32_t n_nodes, const int32_t *path, const int32_t *n_acc,
                                   int32_t max_path, int32_t *status_out, void *stream) {
    if (!ctx || !cache) return READER_ERR_INVALID_ARG;
    if (batch == 0) return READER_OK;
    if (!k_tree || !v_tree || !path || !n_acc || !status_out || !cache->k || !cache->v || !cache->valid || !cache->extent)
        return READER_ERR_INVALID_ARG;
    if (batch < 0 || n_nodes < 1 || n_nodes > kMaxNodes || max_path < 1 || cache->n_kv_heads < 1 || cache->capacity < 1)
        return READER_ERR_INVALID_ARG;
    if (cache->head_dim % 8 != 0 || cache->head_dim < 8) return READER_ERR_UNSUPPORTED;
    if (!aligned16(k_tree) || !aligned16(v_tree) || !aligned16(cache->k) || !aligned16(cache->v)) return READER_ERR_INVALID_ARG;
    if (reader_status st = check_device(ctx)) return st;
    launch_padded_append(static_cast<__nv_bfloat16 *>(cache->k), static_cast<__nv_bfloat16 *>(cache->v), batch,
                         cache->n_kv_heads, cache->capacity, cache->head_dim, cache->valid, cache->extent,
                         static_cast<const __nv_bfloat16 *>(k_tree), static_cast<const __nv_bfloat16 *>(v_tree), n_nodes,
                         path, n_acc, max_path, status_out, (cudaStream_t)stream);
    return launch_status();
}

reader_status reader_padded_rearrange(reader_ctx *ctx, reader_padded_cache *cache, int32_t batch, int32_t *lengths_out,
                                      void *stream) {
    if (!ctx || !cache) return READER_ERR_INVALID_ARG;
    if (batch == 0) return READER_OK;
    if (!cache->extent || !lengths_out) return READER_ERR_INVALID_ARG;
    const reader_status s = reader_kv_rearrange(ctx, cache->k, cache->v, batch, cache->n_kv_heads, cache->capacity,
                                                cache->head_dim, cache->valid, lengths_out, stream);
    if (s != READER_OK) return s;
    launch_set_extent(lengths_out, batch, cache->extent, (cudaStream_t)stream);
    return launch_status();
}

reader_status reader_accept(reader_ctx *ctx, const reader_tree *tree, const int32_t *node_tokens,
                            const float *logits, int32_t vocab, int32_t *target_ids, int32_t max_path,
                            int32_t *path_out, int32_t *n_acc_out, int32_t *bonus_out, void *workspace,
                            size_t workspace_bytes, int32_t *status_out, void *stream) {
    if (!ctx || !tree) return READER_ERR_INVALID_ARG;
    if (tree->batch == 0) return READER_OK;
    if (!tree->parent || !node_tokens || !target_ids || !path_out || !n_acc_out || !bonus_out || !status_out)
        return READER_ERR_INVALID_ARG;
    const int B = tree->batch, T = tree->n_nodes;
    if (B < 0 || T < 1 || T > kMaxNodes || max_path < 1) return READER_ERR_INVALID_ARG;
    if (reader_status st = check_device(ctx)) return st;
    cudaStream_t st = (cudaStream_t)stream;
    int splits = 0;
    float *pv = nullptr;
    int32_t *pi = nullptr;
    if (logits) {
        if (vocab < 1 || !workspace || !aligned16(logits) || (reinterpret_cast<uintptr_t>(workspace) % kAlign) != 0)
            return READER_ERR_INVALID_ARG;
        // only the argmax regions are used, so any head shape that sized the workspace will do
        const WsLayout w = ws_layout(ctx, B, T, 64);
        if (workspace_bytes < w.total) return READER_ERR_WORKSPACE;
        const int64_t rows = (int64_t)B * T;
        splits = argmax_splits(ctx->n_sm, rows, vocab);
        unsigned char *ws = static_cast<unsigned char *>(workspace);
        pv = reinterpret_cast<float *>(ws + w.amax_val);
        pi = reinterpret_cast<int32_t *>(ws + w.amax_idx);
        if (ctx->ev_acc_start) cudaEventRecord(ctx->ev_acc_start, st);
        launch_argmax(logits, rows, vocab, splits, pv, pi, st);
        if (ctx->ev_acc_stop) cudaEventRecord(ctx->ev_acc_stop, st);
    }
    launch_accept(tree->parent, node_tokens, target_ids, B, T, max_path, pv, pi, splits, path_out, n_acc_out,
                  bonus_out, status_out, st);
    return launch_status();
}

reader_status reader_accept_commit(reader_ctx *ctx, const reader_tree *tree, const int32_t *node_tokens, const float *logits,
                                   int32_t vocab, int32_t *target_ids, int32_t max_path, reader_kv_cache *cache,
                                   const void *k_tree, const void *v_tree, int32_t update_seq_lens, int32_t *path_out,
                                   int32_t *n_acc_out, int32_t *bonus_out, int32_t *slots_out, void *workspace,
                                   size_t workspace_bytes, int32_t *status_out, int32_t *commit_status_out, void *stream) {
    if (!ctx || !tree || !cache) return READER_ERR_INVALID_ARG;
    if (tree->batch == 0) return READER_OK;
    if (!tree->parent || !node_tokens || !target_ids || !path_out || !n_acc_out || !bonus_out || !slots_out || !status_out ||
        !commit_status_out || !k_tree || !v_tree || !cache->k_pool || !cache->v_pool || !cache->page_table || !cache->seq_lens)
        return READER_ERR_INVALID_ARG;
    const int B = tree->batch, T = tree->n_nodes;
    if (B < 0 || T < 1 || T > kMaxNodes || max_path < 1 || cache->n_kv_heads < 1 || cache->max_pages_per_seq < 1 ||
        cache->num_pages < 0 || cache->shared_prefix_len < 0 || cache->shared_prefix_len % kPage != 0)
        return READER_ERR_INVALID_ARG;
    if (cache->page_size != kPage || cache->head_dim % 8 != 0 || cache->head_dim < 8) return READER_ERR_UNSUPPORTED;
    if (!aligned16(k_tree) || !aligned16(v_tree) || !aligned16(cache->k_pool) || !aligned16(cache->v_pool))
        return READER_ERR_INVALID_ARG;
    if (reader_status st = check_device(ctx)) return st;
    cudaStream_t st = (cudaStream_t)stream;
    int splits = 0;
    float *pv = nullptr;
    int32_t *pi = nullptr;
    if (logits) {
        if (vocab < 1 || !workspace || !aligned16(logits) || (reinterpret_cast<uintptr_t>(workspace) % kAlign) != 0)
            return READER_ERR_INVALID_ARG;
        const WsLayout w = ws_layout(ctx, B, T, 64);
        if (workspace_bytes < w.total) return READER_ERR_WORKSPACE;
        splits = argmax_splits(ctx->n_sm, (int64_t)B * T, vocab);
        unsigned char *ws = static_cast<unsigned char *>(workspace);
        pv = reinterpret_cast<float *>(ws + w.amax_val);
        pi = reinterpret_cast<int32_t *>(ws + w.amax_idx);
        if (ctx->ev_acc_start) cudaEventRecord(ctx->ev_acc_start, st);
        launch_argmax(logits, (int64_t)B * T, vocab, splits, pv, pi, st);
        if (ctx->ev_acc_stop) cudaEventRecord(ctx->ev_acc_stop, st);
    }
    launch_accept_commit(tree->parent, node_tokens, target_ids, B, T, max_path, pv, pi, splits, path_out, n_acc_out, bonus_out,
                         status_out, *cache, static_cast<const __nv_bfloat16 *>(k_tree), static_cast<const __nv_bfloat16 *>(v_tree),
                         update_seq_lens, slots_out, commit_status_out, st);
    return launch_status();
}

reader_status reader_kv_commit_layers(reader_ctx *ctx, const reader_kv_cache *caches, const void *const *k_trees,
                                      const void *const *v_trees, int32_t n_layers, int32_t batch, int32_t n_nodes,
                                      const int32_t *path, const int32_t *n_acc, int32_t max_path,
                                      int32_t update_seq_lens, int32_t *slots_out, int32_t *status_out, void *stream) {
    if (!ctx || !caches || n_layers < 1) return READER_ERR_INVALID_ARG;
    if (batch == 0) return READER_OK;
    if (!k_trees || !v_trees || !path || !n_acc || !slots_out || !status_out) return READER_ERR_INVALID_ARG;
    const reader_kv_cache &c0 = caches[0];
    if (batch < 0 || n_nodes < 1 || n_nodes > kMaxNodes || max_path < 1 || c0.n_kv_heads < 1 || !c0.page_table ||
        !c0.seq_lens || c0.max_pages_per_seq < 1 || c0.num_pages < 0 || c0.shared_prefix_len < 0 ||
        c0.shared_prefix_len % kPage != 0)
        return READER_ERR_INVALID_ARG;
    if (c0.page_size != kPage || c0.head_dim % 8 != 0 || c0.head_dim < 8) return READER_ERR_UNSUPPORTED;
    std::vector<CommitLayers> chunks((n_layers + kCommitLayersPerLaunch - 1) / kCommitLayersPerLaunch);
    for (int l = 0; l < n_layers; ++l) {
        const reader_kv_cache &c = caches[l];
        if (c.page_table != c0.page_table || c.seq_lens != c0.seq_lens || c.num_pages != c0.num_pages ||
            c.n_kv_heads != c0.n_kv_heads || c.head_dim != c0.head_dim || c.page_size != c0.page_size ||
            c.max_pages_per_seq != c0.max_pages_per_seq || c.shared_prefix_len != c0.shared_prefix_len ||
            !c.k_pool || !c.v_pool || !k_trees[l] || !v_trees[l] || !aligned16(c.k_pool) || !aligned16(c.v_pool) ||
            !aligned16(k_trees[l]) || !aligned16(v_trees[l]))
            return READER_ERR_INVALID_ARG;
        CommitLayers &ch = chunks[l / kCommitLayersPerLaunch];
        const int at = l % kCommitLayersPerLaunch;
        ch.k_pool[at] = static_cast<__nv_bfloat16 *>(c.k_pool);
        ch.v_pool[at] = static_cast<__nv_bfloat16 *>(c.v_pool);
        ch.k_tree[at] = static_cast<const __nv_bfloat16 *>(k_trees[l]);
        ch.v_tree[at] = static_cast<const __nv_bfloat16 *>(v_trees[l]);
    }
    if (reader_status st = check_device(ctx)) return st;
    launch_kv_commit_layers(c0, chunks.data(), n_layers, batch, n_nodes, path, n_acc, max_path, update_seq_lens,
                            slots_out, status_out, (cudaStream_t)stream);
    return launch_status();
}

reader_status reader_kv_rearrange(reader_ctx *ctx, void *k, void *v, int32_t batch, int32_t n_kv_heads,
                                  int32_t capacity, int32_t head_dim, uint8_t *valid, int32_t *lengths_out,
                                  void *stream) {
    if (!ctx) return READER_ERR_INVALID_ARG;
    if (batch == 0) return READER_OK;
    if (!k || !v || !valid || !lengths_out || batch < 0 || n_kv_heads < 1 || capacity < 1 || !aligned16(k) || !aligned16(v))
        return READER_ERR_INVALID_ARG;
    if (head_dim < 8 || head_dim % 8 != 0 || head_dim > 256) return READER_ERR_UNSUPPORTED;   // a chunk of at least 64 rows is staged in 40 KB
    if (reader_status st = check_device(ctx)) return st;
    launch_kv_rearrange(static_cast<__nv_bfloat16 *>(k), static_cast<__nv_bfloat16 *>(v), batch, n_kv_heads, capacity,
                        head_dim, valid, lengths_out, (cudaStream_t)stream);
    return launch_status();
}

reader_status reader_sample_targets(reader_ctx *ctx, const reader_tree *tree, const float *logits, int32_t vocab,
                                    const float *uniforms, float temperature, int32_t top_k, float top_p,
                                    int32_t *target_ids, void *stream) {
    if (!ctx || !tree) return READER_ERR_INVALID_ARG;
    if (tree->batch == 0) return READER_OK;
    if (!tree->parent || !logits || !uniforms || !target_ids || !aligned16(logits)) return READER_ERR_INVALID_ARG;
    const int B = tree->batch, T = tree->n_nodes;
    if (B < 0 || T < 1 || T > kMaxNodes || vocab < 1 || top_k < 0 || !(top_p > 0.f) || !(temperature > 0.f) || temperature > 3.0e38f)
        return READER_ERR_INVALID_ARG;
    if (vocab > sample_max_vocab()) return READER_ERR_UNSUPPORTED;
    if (reader_status st = check_device(ctx)) return st;
    const float c = (float)(1.4426950408889634 / (double)temperature);
    launch_sample(logits, (int64_t)B * T, vocab, tree->parent, uniforms, T, c, top_k, top_p, target_ids, ctx->n_sm, (cudaStream_t)stream);
    return launch_status();
}

reader_status reader_kv_commit(reader_ctx *ctx, reader_kv_cache *cache, const void *k_tree, const void *v_tree,
                               int32_t batch, int32_t n_nodes, const int32_t *path, const int32_t *n_acc,
                               int32_t max_path, int32_t update_seq_lens, int32_t *slots_out, int32_t *status_out,
                               void *stream) {
    if (!ctx || !cache) return READER_ERR_INVALID_ARG;
    if (batch == 0) return READER_OK;
    if (!k_tree || !v_tree || !path || !n_acc || !slots_out || !status_out ||
        !cache->k_pool || !cache->v_pool || !cache->page_table || !cache->seq_lens)
        return READER_ERR_INVALID_ARG;
    if (batch < 0 || n_nodes < 1 || n_nodes > kMaxNodes || max_path < 1 || cache->n_kv_heads < 1 ||
        cache->max_pages_per_seq < 1 || cache->num_pages < 0 || cache->shared_prefix_len < 0 ||
        cache->shared_prefix_len % kPage != 0)
        return READER_ERR_INVALID_ARG;
    if (cache->page_size != kPage || cache->head_dim % 8 != 0 || cache->head_dim < 8) return READER_ERR_UNSUPPORTED;
    if (!aligned16(k_tree) || !aligned16(v_tree) || !aligned16(cache->k_pool) || !aligned16(cache->v_pool))
        return READER_ERR_INVALID_ARG;
    if (reader_status st = check_device(ctx)) return st;
    launch_kv_commit(*cache, static_cast<const __nv_bfloat16 *>(k_tree), static_cast<const __nv_bfloat16 *>(v_tree),
                     batch, n_nodes, path, n_acc, max_path, update_seq_lens, slots_out, status_out,
                     (cudaStream_t)stream);
    return launch_status();
}

}  // extern "C"
