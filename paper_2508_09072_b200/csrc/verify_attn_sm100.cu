// Tree-masked verify attention (Sec. 3.2) on the sm_100a tensor cores.
//
// Two persistent CTAs per SM each walk their range of the flattened split-KV tile list (the CTAs of
// one lane walk the same KV stream, one M tile each: see the work partition in common.cuh).  For
// every unit (sequence, KV head, 128 query rows) a CTA computes S = Q K^T and O += P V with
// tcgen05.mma, one KV tile of 64 keys (one cache page, or 64 tree nodes) at a time:
//
//   warp 8      producer: K tiles and V tiles travel through two separate rings (3 and 2 slots).
//               Every tile arrives by TMA (64x64 boxes, 128-byte swizzle): cache pages from the
//               pool (with an L2 evict-first hint when no other CTA will read them again), tree
//               tiles from the tree tensors, the 128 query rows of the next segment (node j, group
//               member g -> row j*G+g) by one 4-D box per 64 columns as soon as the previous
//               segment's last score product is done.  A K slot is free again as soon as its score
//               product has run, long before the tile's value product, so key loads run far ahead.
//   warp 9      issues S[i] = Q K[i]^T as soon as K[i] has landed and the score tile is free
//   warp 10     issues O += P[j] V[j] as soon as P[j] and V[j] are ready.  Both issuers (and the producer)
//               issue from the lane elect.sync picks: under `if (lane == 0)` one tcgen05.mma started
//               only every 110-160 cycles, behind elect.sync one starts every 48-64.
//   warps 0-7   softmax: warp w owns the 16 query rows 32 (w % 4) + 16 (w / 4) .. + 15 (TMEM lanes), a
//               quad of threads per row pair (rows r and r + 8), so a thread handles 16 of a row's 64
//               scores and a row's maximum costs two shuffles (paid only when it rises: the vote on that
//               uses the threads' own maxima).  Scores come from TMEM, the ancestor
//               bitmask / length mask is applied, the running maximum is raised only when it grows
//               by more than 2^8 (the accumulator in TMEM is rescaled then), probabilities (bf16
//               pairs) go to one of two probability tiles in TMEM and are the value product's A
//               operand straight from there.  The same threads write O (or an (m, l, O) partial) at
//               the end of a segment.
//
// The same kernel has a second form (kSmall) for calls with few units, launched alone: one thread-block
// cluster per unit whose CTAs check the sequence, share the unit's tiles and merge their shares after the
// cluster's hardware barrier (see where kSmall is tested below).
//
// Bytes beyond a sequence's length or the tree's end can never reach a product: scores there are
// replaced by -inf, and the value product skips 16-key slices past the end and zeroes the tail of
// the last slice in shared memory first.
//
// TMEM: columns 0-63 hold the score tile S (fp32), columns 64-127 two probability tiles P (32 columns
// each: bf16 pairs), columns 128.. hold O (head_dim columns, fp32); lane = query row.  S is free again as
// soon as the softmax warps hold it in registers, so the score product of tile i+1 runs beside the softmax
// of tile i; P[i & 1] is free once the value product of tile i has read it, two tiles before it is
// written again.  (With P written over its scores in one of two 64-column buffers, the score product of
// tile i+1 had to wait for the value product of tile i-1: issue of four value MMAs, issue of eight score
// MMAs and the softmax sat on one dependency chain per buffer, 1670 cycles per tile of which the tensor
// pipe worked 45 %.)
//
// Barriers: a parity wait can only tell a barrier's current phase from the one before it.  s_full / s_empty
// alternate strictly (the score product of tile i+1 needs every softmax thread's arrival for tile i, which
// comes after that thread saw tile i), so one barrier each is enough; p_full and pv_done, which warps
// reach at different times, exist once per probability tile: the waiter for tile i on barrier i & 1 knows
// that tile i-2 is complete and that tile i+2 cannot have been issued.  Every wait is bounded: after one
// second without progress a CTA raises the error flag in the workspace, stops waiting and runs to its end.
#include <cuda.h>

#include <new>

#include "ptx_sm100.cuh"
#include "tree.cuh"
#include "verify_attn_sm100.cuh"

namespace reader {
namespace {

using namespace ptx;

constexpr int kStagesK = 3;         // K tiles in flight per CTA (two CTAs share an SM)
constexpr int kStagesV = 2;         // V tiles
constexpr int kSoftmaxWarps = 8;   // 16 query rows each
constexpr int kThreads = (kSoftmaxWarps + 3) * 32;
constexpr int kProducerWarp = kSoftmaxWarps;
constexpr int kMmaWarp = kSoftmaxWarps + 1;   // issues the score products, owns the TMEM allocation
constexpr int kPvWarp = kSoftmaxWarps + 2;    // issues the value products
constexpr uint64_t kWaitLimitNs = 1000000000ull;
constexpr float kRaiseMaxBy = 8.f;   // log2 units
constexpr uint32_t kTmemCols = 256;
constexpr uint32_t kTmemS = 0;      // the score tile (64 columns, fp32)
constexpr uint32_t kTmemP = 64;     // two probability tiles (32 columns each: bf16 pairs)
constexpr uint32_t kTmemO = 128;    // the output accumulator (head_dim columns, fp32)

template <int D>
struct Cfg {
    static constexpr int kHalves = D / 64;                 // 64-column (128-byte) blocks per row
    static constexpr int kHalfRowsQ = kTileM * 128;        // bytes of one 64-column block of Q
    static constexpr int kHalfRowsKV = kPage * 128;        // bytes of one 64-column block of a KV tile
    static constexpr int kQBytes = kTileM * D * 2;
    static constexpr int kTileBytes = kPage * D * 2;
    static constexpr int kOffQ = 0;
    static constexpr int kOffK = kQBytes;                          // ring of K tiles
    static constexpr int kOffV = kOffK + kStagesK * kTileBytes;    // ring of V tiles
    static constexpr int kOffBars = kOffV + kStagesV * kTileBytes;
    static constexpr int kSmemBytes = kOffBars + 256;   // + barriers; two CTAs of head_dim 128 fit one SM
    // the single-launch kernel for small calls also keeps one sequence's parent array there
    static constexpr int kOffParents = kOffBars + 256;
    static constexpr int kSmemBytesSmall = kOffParents + kMaxNodes * 4;
};

struct Bars {
    uint64_t k_full[kStagesK], k_empty[kStagesK], v_full[kStagesV], v_empty[kStagesV];
    uint64_t q_full, q_empty, s_full, s_empty, p_full[2], pv_done[2];
    uint32_t tmem_base;
    int32_t abort;
    int32_t reject;   // small-call kernel: status code of a sequence the checks turned down
};
static_assert(sizeof(Bars) <= 256, "barrier block");

// Bounded wait.  Returns false when the CTA has given up.
__device__ __forceinline__ bool wait(uint32_t bar, uint32_t parity, volatile int32_t *abort_s, int32_t *error_flag) {
    if (mbar_try_wait(bar, parity)) return true;
    if (*abort_s) return false;
    const uint64_t t0 = globaltimer_ns();
    while (true) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort_s) return false;
        if (globaltimer_ns() - t0 > kWaitLimitNs) {
            *abort_s = 1;
            atomicExch(error_flag, (int32_t)READER_ERR_TIMEOUT);
            return false;
        }
    }
}


// Gives up after kWaitLimitNs without progress in a polling loop.
struct Watchdog {
    uint64_t t0 = 0;
    bool armed = false;
    __device__ __forceinline__ void progress() { armed = false; }
    __device__ __forceinline__ bool expired(volatile int32_t *abort_s, int32_t *error_flag) {
        if (*abort_s) return true;
        if (!armed) {
            armed = true;
            t0 = globaltimer_ns();
            return false;
        }
        if (globaltimer_ns() - t0 > kWaitLimitNs) {
            *abort_s = 1;
            atomicExch(error_flag, (int32_t)READER_ERR_TIMEOUT);
            return true;
        }
        return false;
    }
};

// Warp-uniform, non-blocking test of an mbarrier phase (true only once every lane has seen it).
__device__ __forceinline__ bool ready(uint32_t bar, uint32_t parity) {
    return __all_sync(0xffffffffu, mbar_test_wait(bar, parity));
}

// The cache kind is a compile-time choice (kPadded: the padded batch cache of Sec. 4.3, else the paged
// cache), so that neither pays for the other's addressing.
template <bool kPadded>
__device__ __forceinline__ uint64_t visible_of(const AttnParams &p, int b, int t, int L) {
    if constexpr (kPadded) {
        return p.valid_bits[(size_t)b * p.bits_per_seq + t];
    } else {
        const int valid = L - t * kPage;
        return valid >= kPage ? ~0ull : ((1ull << valid) - 1);
    }
}

// Where a CTA's work comes from.  The general kernel walks a range of the flattened tile list laid out by
// the preparation kernel; the single-launch kernel for small calls (kSmall) has exactly one segment, the
// share of its unit's tiles that its rank in the cluster gives it, and counts flat positions in tiles.
template <bool kSmall, bool kPadded>
__device__ __forceinline__ Segment seg_at(const AttnParams &p, const WarpSched &ws, const Segment &mine, int cta, int w, int w_end,
                                          int lane) {
    if constexpr (kSmall) {
        Segment g = mine;
        g.tile_begin = mine.tile_begin + w;
        g.span = w_end - w;
        return g;
    } else {
        return segment_at_warp(p.sched, ws, kPadded ? nullptr : p.seq_lens, p.B, cta, w, w_end, lane);
    }
}

// Walks the tiles of a CTA's range in order; the producer keeps one cursor for keys and one for
// values.  Page ids are fetched 32 at a time (one per lane) and handed out by shuffle.
template <bool kPadded, bool kSmall>
struct TileCursor {
    int w, w_end;       // flat position of the next segment
    Segment sg, mine;
    int L;              // committed length of sg.b
    int t;              // current tile within the unit
    int it;             // tiles handed out so far
    int cache_t0, cache_page;
    bool active;

    __device__ __forceinline__ void refill(const AttnParams &p, int lane) {
        cache_t0 = t;
        const int tt = t + lane;
        if constexpr (kPadded) cache_page = 0;
        else cache_page = (tt < sg.tile_end && tt < sg.npages) ? p.page_table[(size_t)sg.b * p.max_pages + tt] : 0;
    }
    __device__ __forceinline__ void next_segment(const AttnParams &p, const WarpSched &ws, int cta, int lane) {
        active = false;
        while (w < w_end) {   // segments without a real tile (a range that ends among overhead entries) are skipped
            sg = seg_at<kSmall, kPadded>(p, ws, mine, cta, w, w_end, lane);
            w += sg.span;
            if (sg.tile_end > sg.tile_begin) { active = true; break; }
        }
        if (!active) return;
        L = sg.len;
        t = sg.tile_begin;
        refill(p, lane);
    }
    __device__ __forceinline__ void init(const AttnParams &p, const WarpSched &ws, const Segment &mine_, int cta, int lane, int w_begin,
                                         int w_end_) {
        mine = mine_;
        w = w_begin; w_end = w_end_; it = 0;
        next_segment(p, ws, cta, lane);
    }
    __device__ __forceinline__ int page() const { return __shfl_sync(0xffffffffu, cache_page, t - cache_t0); }
    __device__ __forceinline__ void advance(const AttnParams &p, const WarpSched &ws, int cta, int lane) {
        ++t; ++it;
        if (t == sg.tile_end) next_segment(p, ws, cta, lane);
        else if (t - cache_t0 == 32) refill(p, lane);
    }
};

// One K or V tile into its ring slot, always by TMA: a cache page comes whole from the pool (the
// page exists in full even when the sequence ends inside it), a tree tile comes as 64 node rows of
// one KV head from the tree tensor (rows past the tensor's end read as zero).  Rows past the
// valid count may therefore hold anything; the score side masks them by selection and the value
// side never multiplies them (see the MMA issuer).  Called by the whole producer warp.
template <int D, bool kPadded, bool kSmall>
__device__ __forceinline__ void load_tile(const AttnParams &p, const TileCursor<kPadded, kSmall> &c, const CUtensorMap *pool_map,
                                          const CUtensorMap *tree_map, uint32_t dst, uint32_t full, int lane,
                                          uint64_t stream_policy, int first_streamed_tile) {
    using C = Cfg<D>;
    const int page = c.page();
    __syncwarp();
    if (!elect_one()) return;   // (as for the MMA issuers: behind elect.sync the copies are issued back to back)
    mbar_arrive_expect_tx(full, C::kTileBytes);
    if (c.t < c.sg.npages) {
        int row;
        if constexpr (kPadded) row = (c.sg.b * p.Hkv + c.sg.h) * p.cap + c.t * kPage;
        else row = (page * p.Hkv + c.sg.h) * kPage;
#pragma unroll
        for (int hf = 0; hf < C::kHalves; ++hf) {
            // a page that no other CTA will read again should not push reusable lines out of L2
            if (c.t >= first_streamed_tile) tma_load_2d_hint(dst + hf * C::kHalfRowsKV, pool_map, full, hf * 64, row, stream_policy);
            else tma_load_2d(dst + hf * C::kHalfRowsKV, pool_map, full, hf * 64, row);
        }
    } else {
        const int node0 = c.sg.b * p.T + (c.t - c.sg.npages) * kPage;
#pragma unroll
        for (int hf = 0; hf < C::kHalves; ++hf) tma_load_3d(dst + hf * C::kHalfRowsKV, tree_map, full, hf * 64, c.sg.h, node0);
    }
}

template <int D, bool kPadded, bool kSmall>
__global__ void __launch_bounds__(kThreads, 2)
attn_sm100_kernel(const AttnParams p, const __grid_constant__ CUtensorMap kmap, const __grid_constant__ CUtensorMap vmap,
                  const __grid_constant__ CUtensorMap ktmap, const __grid_constant__ CUtensorMap vtmap,
                  const __grid_constant__ CUtensorMap qmap) {
    using C = Cfg<D>;
    extern __shared__ __align__(1024) unsigned char smem[];
    const uint32_t base = smem_u32(smem);
    if (base & 1023u) {   // the swizzled tiles need 1024-byte alignment; never seen, but checked
        if (threadIdx.x == 0) atomicExch(p.error_flag, (int32_t)READER_ERR_CUDA);
        return;
    }
    Bars *bars = reinterpret_cast<Bars *>(smem + C::kOffBars);
    volatile int32_t *abort_s = &bars->abort;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int cta = blockIdx.x;

    const uint32_t sQ = base + C::kOffQ, sK = base + C::kOffK, sV = base + C::kOffV;
    auto bar = [&](const uint64_t *b) { return smem_u32(b); };

    if (tid == 0) {
        for (int s = 0; s < kStagesK; ++s) {
            mbar_init(bar(&bars->k_full[s]), 1);
            mbar_init(bar(&bars->k_empty[s]), 1);
        }
        for (int s = 0; s < kStagesV; ++s) {
            mbar_init(bar(&bars->v_full[s]), 1);
            mbar_init(bar(&bars->v_empty[s]), 1);
        }
        mbar_init(bar(&bars->q_full), 1);
        mbar_init(bar(&bars->q_empty), 1);
        mbar_init(bar(&bars->s_full), 1);
        mbar_init(bar(&bars->s_empty), kSoftmaxWarps * 32);
        mbar_init(bar(&bars->p_full[0]), kSoftmaxWarps * 32);
        mbar_init(bar(&bars->p_full[1]), kSoftmaxWarps * 32);
        mbar_init(bar(&bars->pv_done[0]), 1);
        mbar_init(bar(&bars->pv_done[1]), 1);
        bars->abort = 0;
        bars->reject = 0;
        fence_mbar_init();
        fence_proxy_async();
    }
    if (warp == kMmaWarp) {
        tmem_alloc(smem_u32(&bars->tmem_base), kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = bars->tmem_base;

    // everything above overlapped the kernel before this one in the stream; its results are read from here on
    grid_dependency_wait();
    grid_launch_dependents();
    WarpSched wsched{0x7fffffff, 0, 0, 0};
    CtaWork cw{0, 0, 0, 0};
    Segment mine{};          // kSmall: this CTA's share of its unit
    int W = 0, w_begin = 0, w_end = 0;
    int reject = 0;          // kSmall: status code of a sequence the checks below turn down
    uint32_t cl_rank = 0, cl_size = 1;
    const int32_t *par = reinterpret_cast<const int32_t *>(smem + C::kOffParents);   // kSmall only
    if constexpr (kSmall) {
        // One launch does everything for a call with few units: the cluster (b, KV head, M tile) checks its
        // sequence itself (what the preparation kernel does for large calls), cuts the unit's tiles into one
        // share per CTA of the cluster, and merges the shares (partials in the workspace, ordered by the
        // cluster's hardware barrier) at the end.
        cl_rank = cluster_ctarank();
        cl_size = cluster_nctarank();
        const int n_mtiles = (p.T * p.G + kTileM - 1) / kTileM;
        const int unit = cta / (int)cl_size;
        mine.mt = unit % n_mtiles;
        mine.h = (unit / n_mtiles) % p.Hkv;
        mine.b = unit / (n_mtiles * p.Hkv);
        // Only the committed length is needed to start loading: the checks of the tree and of the page ids run
        // in the softmax warps (below) while the first tiles are on their way, and their outcome is used at the
        // end.  (A page id outside the pool makes a tile load read the fill value, never a fault.)
        const int L = p.seq_lens[mine.b];
        const bool len_ok = L >= 0 && (int64_t)L <= (int64_t)p.max_pages * kPage;
        const bool flagged = p.zero_rejected && *p.error_flag != 0;   // a layer call after a layer that gave up a wait
        const int npages = (len_ok && !flagged) ? (L + kPage - 1) / kPage : 0;
        const int n = (len_ok && !flagged) ? npages + (p.T + kPage - 1) / kPage : 0;
        mine.ntiles = n;
        mine.npages = npages;
        mine.len = L;
        mine.tile_begin = mul_div((int)cl_rank, n, (int)cl_size);
        mine.tile_end = mul_div((int)cl_rank + 1, n, (int)cl_size);
        mine.full = cl_size == 1;
        mine.slot = cta;
        w_end = mine.tile_end - mine.tile_begin;
        if (tid == 0) {
            if (flagged) atomicOr(&bars->reject, 8);
            else if (!len_ok) atomicOr(&bars->reject, 2);
        }
    } else {
        wsched = load_warp_sched(p.sched, kPadded ? nullptr : p.seq_lens, p.B, lane);   // in flight with W
        W = p.sched.seq_tile_start[p.B];
        cw = cta_work(p.sched, p.B, cta, W);
        w_begin = cw.w_begin;
        w_end = cw.w_end;
    }

    if (warp == kProducerWarp) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            prefetch_tensormap(&kmap);
            prefetch_tensormap(&vmap);
            prefetch_tensormap(&ktmap);
            prefetch_tensormap(&vtmap);
            prefetch_tensormap(&qmap);
        }
        // pages are read exactly once when a KV head has a single M tile, except those of a shared prefix, which
        // the other sequences' CTAs will ask for again: the hint goes on the private pages only
        const uint64_t stream_policy = l2_policy_evict_first();
        const int first_streamed_tile = p.sched.n_mtiles == 1 ? p.shared_prefix_pages : 0x7fffffff;
        TileCursor<kPadded, kSmall> kc, vc;
        kc.init(p, wsched, mine, cta, lane, w_begin, w_end);
        vc.init(p, wsched, mine, cta, lane, w_begin, w_end);
        // the query tile of the next segment goes in as soon as the last score product of the
        // current one has retired (Q is single-buffered)
        int q_w = w_begin, q_seg = 0;
        const int rows_per_node_tile = kTileM / p.G;
        Watchdog dog;
        while (kc.active || vc.active || q_w < w_end) {
            bool moved = false;
            if (q_w < w_end && ready(bar(&bars->q_empty), (q_seg & 1) ^ 1)) {
                const Segment sg = seg_at<kSmall, kPadded>(p, wsched, mine, cta, q_w, w_end, lane);
                q_w += sg.span;
                if (sg.tile_end <= sg.tile_begin) continue;   // no real tile: no query tile
                __syncwarp();
                if (elect_one()) {
                    const uint32_t full = bar(&bars->q_full);
                    mbar_arrive_expect_tx(full, C::kQBytes);
#pragma unroll
                    for (int hf = 0; hf < C::kHalves; ++hf)
                        tma_load_4d(sQ + hf * C::kHalfRowsQ, &qmap, full, hf * 64, sg.h * p.G, sg.mt * rows_per_node_tile, sg.b);
                }
                __syncwarp();
                ++q_seg;
                moved = true;
            }
            if (kc.active) {
                const int stage = kc.it % kStagesK;
                if (ready(bar(&bars->k_empty[stage]), ((kc.it / kStagesK) & 1) ^ 1)) {
                    load_tile<D, kPadded, kSmall>(p, kc, &kmap, &ktmap, sK + stage * C::kTileBytes, bar(&bars->k_full[stage]), lane, stream_policy, first_streamed_tile);
                    __syncwarp();
                    kc.advance(p, wsched, cta, lane);
                    moved = true;
                }
            }
            if (vc.active) {
                const int stage = vc.it % kStagesV;
                if (ready(bar(&bars->v_empty[stage]), ((vc.it / kStagesV) & 1) ^ 1)) {
                    load_tile<D, kPadded, kSmall>(p, vc, &vmap, &vtmap, sV + stage * C::kTileBytes, bar(&bars->v_full[stage]), lane, stream_policy, first_streamed_tile);
                    __syncwarp();
                    vc.advance(p, wsched, cta, lane);
                    moved = true;
                }
            }
            if (moved) dog.progress();
            else if (dog.expired(abort_s, p.error_flag)) break;
        }
        // a CTA that gave up must not exit under its own copies: let the last ones land (bounded)
        if (*abort_s) {
            const uint64_t t0 = globaltimer_ns();
            for (int i = max(0, kc.it - kStagesK); i < kc.it; ++i)
                while (!mbar_try_wait(bar(&bars->k_full[i % kStagesK]), (i / kStagesK) & 1) && globaltimer_ns() - t0 < 20000000ull) {
                }
            for (int i = max(0, vc.it - kStagesV); i < vc.it; ++i)
                while (!mbar_try_wait(bar(&bars->v_full[i % kStagesV]), (i / kStagesV) & 1) && globaltimer_ns() - t0 < 20000000ull) {
                }
        }
    } else if (warp == kMmaWarp) {
        // ------------------------------------------------------------------ score-product issuer
        // (its own warp, so that a tile's value product never queues behind the next tile's score product)
        constexpr uint32_t kIdescQK = idesc_bf16_f32(kTileM, kPage, false, false);
        // descriptors differ only in their start-address field (bytes >> 4), so each operand's
        // descriptor is one addition away from a base built once
        const uint64_t descQ = smem_desc_sw128(sQ, 16, 1024), descK = smem_desc_sw128(sK, 16, 1024);
        int i = 0, seg = 0;
        int w = w_begin;
        while (w < w_end && !*abort_s) {
            const Segment sg = seg_at<kSmall, kPadded>(p, wsched, mine, cta, w, w_end, lane);
            const int n = sg.tile_end - sg.tile_begin;
            w += sg.span;
            if (n <= 0) continue;
            wait(bar(&bars->q_full), seg & 1, abort_s, p.error_flag);
            for (int t = 0; t < n; ++t, ++i) {
                const int stage = i % kStagesK;
                wait(bar(&bars->k_full[stage]), (i / kStagesK) & 1, abort_s, p.error_flag);
                // the score tile is free as soon as every softmax thread holds the previous scores in registers
                wait(bar(&bars->s_empty), (i & 1) ^ 1, abort_s, p.error_flag);
                tc_fence_after();
                __syncwarp();
                if (elect_one()) {
                    const uint64_t kd = descK + (uint64_t)((stage * C::kTileBytes) >> 4);
#pragma unroll
                    for (int hf = 0; hf < C::kHalves; ++hf)
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk)
                            mma_bf16_ss(tmem + kTmemS, descQ + (uint64_t)((hf * C::kHalfRowsQ + kk * 32) >> 4),
                                        kd + (uint64_t)((hf * C::kHalfRowsKV + kk * 32) >> 4), kIdescQK, (hf | kk) != 0);
                    mma_commit(bar(&bars->k_empty[stage]));
                    mma_commit(bar(&bars->s_full));
                    if (t == n - 1) mma_commit(bar(&bars->q_empty));
                }
                __syncwarp();
            }
            ++seg;
        }
    } else if (warp == kPvWarp) {
        // ------------------------------------------------------------------ value-product issuer
        constexpr uint32_t kIdescPV = idesc_bf16_f32(kTileM, D, false, true);
        const uint64_t descV = smem_desc_sw128(sV, C::kHalfRowsKV, 1024);
        int i = 0;
        int w = w_begin;
        // This warp also leaves the note the combine kernel needs about a unit this CTA starts without finishing
        // it (at most one per CTA): it has time to spare at the start of a segment, the softmax warps do not.
        // (A CTA that gives up on a wait may skip a note: the combine kernel then reports the timeout instead.)
        if constexpr (!kSmall) {
            if (lane == 0) p.split_desc[cta].b = -1;
            __syncwarp();
        }
        while (w < w_end && !*abort_s) {
            const Segment sg = seg_at<kSmall, kPadded>(p, wsched, mine, cta, w, w_end, lane);
            const int n = sg.tile_end - sg.tile_begin;
            if constexpr (!kSmall) {
                if (lane == 0) record_split(p.split_desc, p.sched, p.B, cw.n_lanes, sg, cta, W);
                __syncwarp();
            }
            w += sg.span;
            if (n <= 0) continue;
            const int L = sg.len;
            uint64_t vis_next = 0;
            if constexpr (kPadded) vis_next = sg.tile_begin < sg.npages ? visible_of<true>(p, sg.b, sg.tile_begin, L) : 0;
            for (int tl = 0; tl < n; ++tl, ++i) {
                const int stage = i % kStagesV;
                const int t = sg.tile_begin + tl;
                const uint32_t vbase = sV + stage * C::kTileBytes;
                int slices;
                if constexpr (kPadded) {
                    // keys no query may see (padding rows anywhere in the tile, nodes past the tree's end) must
                    // not reach the product, whatever bytes they hold: 16-key slices behind the last visible
                    // key are not multiplied at all, invisible rows before it are zeroed in place
                    uint64_t vis = vis_next;
                    if (t >= sg.npages) {
                        const int nodes = min(kPage, p.T - (t - sg.npages) * kPage);
                        vis = nodes >= kPage ? ~0ull : ((1ull << nodes) - 1);
                    }
                    if (t + 1 < sg.tile_end && t + 1 < sg.npages) vis_next = visible_of<true>(p, sg.b, t + 1, L);   // ahead of the waits
                    slices = (64 - __clzll((long long)vis) + 15) >> 4;
                    if (tl == 0 && slices == 0) slices = 1;   // the first product of a segment initialises O
                    const uint64_t zero_rows = ~vis & (slices == 4 ? ~0ull : ((1ull << (slices * 16)) - 1));
                    wait(bar(&bars->p_full[i & 1]), (i >> 1) & 1, abort_s, p.error_flag);
                    wait(bar(&bars->v_full[stage]), (i / kStagesV) & 1, abort_s, p.error_flag);
                    tc_fence_after();
                    if (zero_rows) {
                        constexpr int kChunks = D / 8;              // 16-byte pieces per row
                        constexpr int kRowsPerPass = 32 / kChunks;  // rows a warp zeroes at once
                        uint64_t left = zero_rows;
                        while (left) {
                            // lanes 0..kChunks-1 take the lowest row still to do, the next kChunks lanes the one after
                            uint64_t mine = left;
                            for (int q = 0; q < lane / kChunks && mine; ++q) mine &= mine - 1;
                            if (mine) {
                                const int rr = __ffsll((long long)mine) - 1, cc = lane % kChunks;
                                const uint32_t off = (cc >> 3) * C::kHalfRowsKV + rr * 128 + (((cc & 7) ^ (rr & 7)) << 4);
                                asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(vbase + off), "r"(0u) : "memory");
                            }
                            for (int q = 0; q < kRowsPerPass && left; ++q) left &= left - 1;
                        }
                        fence_proxy_async();
                        __syncwarp();
                    }
                } else {
                    wait(bar(&bars->p_full[i & 1]), (i >> 1) & 1, abort_s, p.error_flag);
                    wait(bar(&bars->v_full[stage]), (i / kStagesV) & 1, abort_s, p.error_flag);
                    tc_fence_after();
                    // keys past the end of the sequence / tree: whole 16-key slices are not multiplied at
                    // all, the rest of the last slice is zeroed in place
                    const int valid = t < sg.npages ? min(kPage, L - t * kPage) : min(kPage, p.T - (t - sg.npages) * kPage);
                    slices = (valid + 15) >> 4;
                    if (valid & 15) {
                        constexpr int kChunks = D / 8;
                        for (int idx = lane; idx < (slices * 16 - valid) * kChunks; idx += 32) {
                            const int rr = valid + idx / kChunks, cc = idx % kChunks;
                            const uint32_t off = (cc >> 3) * C::kHalfRowsKV + rr * 128 + (((cc & 7) ^ (rr & 7)) << 4);
                            asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(vbase + off), "r"(0u) : "memory");
                        }
                        fence_proxy_async();
                        __syncwarp();
                    }
                }
                __syncwarp();
                if (elect_one()) {
                    const uint64_t vd = descV + (uint64_t)((stage * C::kTileBytes) >> 4);
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)
                        if (kk < slices)
                            mma_bf16_ts(tmem + kTmemO, tmem + kTmemP + (i & 1) * 32 + kk * 8, vd + (uint64_t)((kk * 2048) >> 4),
                                        kIdescPV, (tl | kk) != 0);
                    mma_commit(bar(&bars->v_empty[stage]));
                    mma_commit(bar(&bars->pv_done[i & 1]));
                }
                __syncwarp();
            }
        }
    } else if (warp < kSoftmaxWarps) {
        // ------------------------------------------------------------------ softmax / epilogue
        // this thread: rows row_a and row_b = row_a + 8 of the M tile, columns 8u + 2 cpair (+1), u = 0..7
        const int cpair = lane & 3;
        const int row_a = (warp & 3) * 32 + (warp >> 2) * 16 + (lane >> 2), row_b = row_a + 8;
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32 + (warp >> 2) * 16) << 16;
        constexpr uint32_t kNegInf = 0xff800000u;
        int it = 0;
        int w = w_begin;
        const int lg_G = 31 - __clz(p.G);
        bool tree_ok = true;
        if constexpr (kSmall) {
            // the checks the preparation kernel makes for large calls: parent[0] = -1 and 0 <= parent[j] < j; every
            // page id in use inside the pool.  256 threads, then one barrier among the softmax warps.
            int32_t *par_w = reinterpret_cast<int32_t *>(smem + C::kOffParents);
            int bits = 0;
            for (int j = tid; j < p.T; j += kSoftmaxWarps * 32) {
                const int pj = p.parent[(size_t)mine.b * p.T + j];
                par_w[j] = pj;
                if (!(j == 0 ? pj == -1 : (pj >= 0 && pj < j))) bits |= 1;
            }
            for (int i = tid; i < mine.npages; i += kSoftmaxWarps * 32) {
                const int pg = p.page_table[(size_t)mine.b * p.max_pages + i];
                if (pg < 0 || pg >= p.num_pages) bits |= 4;
            }
            if (bits) atomicOr(&bars->reject, bits);
            asm volatile("bar.sync 1, %0;" ::"n"(kSoftmaxWarps * 32) : "memory");
            tree_ok = (*reinterpret_cast<volatile int32_t *>(&bars->reject) & 1) == 0;
        }
        if (kSmall && w_end == 0 && cpair == 0) {
            // no tile fell to this CTA: its share of the unit is the empty partial
            *reinterpret_cast<float2 *>(p.partial_ml + ((size_t)cta * kTileM + row_a) * 2) = make_float2(-INFINITY, 0.f);
            *reinterpret_cast<float2 *>(p.partial_ml + ((size_t)cta * kTileM + row_b) * 2) = make_float2(-INFINITY, 0.f);
        }
        while (w < w_end) {
            const Segment sg = seg_at<kSmall, kPadded>(p, wsched, mine, cta, w, w_end, lane);
            w += sg.span;
            if (sg.tile_end <= sg.tile_begin) continue;
            const int L = sg.len;
            const int grow_a = sg.mt * kTileM + row_a, grow_b = grow_a + 8;
            const bool ok_a = grow_a < p.T * p.G, ok_b = grow_b < p.T * p.G;
            // (G divides 128, so it is a power of two: shifts, not divisions, on the path into a segment)
            const int j_a = ok_a ? grow_a >> lg_G : 0, j_b = ok_b ? grow_b >> lg_G : 0;
            const int hq_a = sg.h * p.G + (ok_a ? grow_a & (p.G - 1) : 0), hq_b = sg.h * p.G + (ok_b ? grow_b & (p.G - 1) : 0);

            // The ancestor masks are fetched when a tree tile comes up (the last one or two tiles of a unit), not
            // kept in eight registers through the committed tiles: the loop below runs at the register ceiling.
            auto tree_mask = [&](int tree_tile, bool ok, int j) -> uint64_t {
                if (!ok) return 0ull;
                if (kSmall && p.anc == nullptr) {   // no encoded masks at hand: walk the parent array (in shared memory)
                    uint64_t lo = 0, hi = 0;
                    int lv;
                    if (tree_ok) node_ancestors(par, p.T, j, lo, hi, lv);
                    return tree_tile ? hi : lo;
                }
                return p.anc[((size_t)sg.b * p.T + j) * 2 + tree_tile];
            };

            float m_a = -INFINITY, m_b = -INFINITY, l_a = 0.f, l_b = 0.f;   // l: this thread's share of the row sums
            for (int t = sg.tile_begin; t < sg.tile_end; ++t, ++it) {
                // (with a padded cache the mask comes from memory: the load is issued ahead of the wait below)
                uint64_t vis_a, vis_b;
                if (t < sg.npages) {
                    vis_a = vis_b = visible_of<kPadded>(p, sg.b, t, L);
                } else {
                    vis_a = tree_mask(t - sg.npages, ok_a, j_a);
                    vis_b = tree_mask(t - sg.npages, ok_b, j_b);
                }
                const int buf = it & 1;
                wait(bar(&bars->s_full), it & 1, abort_s, p.error_flag);
                tc_fence_after();
                uint32_t s[32];
                tmem_ld_16x256b_x8(tmem + lane_base + kTmemS, s);
                tmem_wait_ld();
                // the scores are in registers: the next score product may overwrite the tile
                tc_fence_before();
                mbar_arrive(bar(&bars->s_empty));

                if ((vis_a & vis_b) != ~0ull) {
                    const uint64_t ma = vis_a >> (2 * cpair), mb = vis_b >> (2 * cpair);
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        if (!((ma >> (8 * u)) & 1ull)) s[4 * u + 0] = kNegInf;
                        if (!((ma >> (8 * u + 1)) & 1ull)) s[4 * u + 1] = kNegInf;
                        if (!((mb >> (8 * u)) & 1ull)) s[4 * u + 2] = kNegInf;
                        if (!((mb >> (8 * u + 1)) & 1ull)) s[4 * u + 3] = kNegInf;
                    }
                }
                auto f = [&](int i) { return __uint_as_float(s[i]); };
                // this thread's 16 scores of each row, then the other three threads of the quad
                float xa0 = max3(f(0), f(1), f(4)), xa1 = max3(f(5), f(8), f(9));
                float xb0 = max3(f(2), f(3), f(6)), xb1 = max3(f(7), f(10), f(11));
                xa0 = max3(xa0, f(12), f(13)); xa1 = max3(xa1, f(16), f(17));
                xb0 = max3(xb0, f(14), f(15)); xb1 = max3(xb1, f(18), f(19));
                xa0 = max3(xa0, f(20), f(21)); xa1 = max3(xa1, f(24), f(25));
                xb0 = max3(xb0, f(22), f(23)); xb1 = max3(xb1, f(26), f(27));
                float mx_a = max3(xa0, xa1, fmaxf(f(28), f(29))), mx_b = max3(xb0, xb1, fmaxf(f(30), f(31)));
                // A row's maximum rises (by more than 2^8) exactly if one of its four threads holds such a score, so
                // the vote needs no exchange within the quad; the two shuffle rounds that give the row maxima
                // themselves are paid only by the tiles that do raise one (a segment's first tile always does).
                const bool first = t == sg.tile_begin;
                const bool raise = __any_sync(0xffffffffu, mx_a * p.scale_log2 > m_a + kRaiseMaxBy || mx_b * p.scale_log2 > m_b + kRaiseMaxBy);
                float alpha_a = 1.f, alpha_b = 1.f;
                if (raise || first) {
                    mx_a = fmaxf(mx_a, __shfl_xor_sync(0xffffffffu, mx_a, 1));
                    mx_b = fmaxf(mx_b, __shfl_xor_sync(0xffffffffu, mx_b, 1));
                    mx_a = fmaxf(mx_a, __shfl_xor_sync(0xffffffffu, mx_a, 2));
                    mx_b = fmaxf(mx_b, __shfl_xor_sync(0xffffffffu, mx_b, 2));
                    const float mn_a = fmaxf(m_a, mx_a * p.scale_log2), mn_b = fmaxf(m_b, mx_b * p.scale_log2);
                    alpha_a = (mn_a == -INFINITY) ? 1.f : ex2(m_a - mn_a);
                    alpha_b = (mn_b == -INFINITY) ? 1.f : ex2(m_b - mn_b);
                    m_a = mn_a; m_b = mn_b;
                    l_a *= alpha_a; l_b *= alpha_b;
                }
                // packed fp32x2 arithmetic: one instruction scales two scores, one adds two probabilities
                const float2 sc2 = make_float2(p.scale_log2, p.scale_log2);
                const float nma = (m_a == -INFINITY) ? 0.f : -m_a, nmb = (m_b == -INFINITY) ? 0.f : -m_b;
                const float2 nma2 = make_float2(nma, nma), nmb2 = make_float2(nmb, nmb);
                float2 lsa = make_float2(0.f, 0.f), lsb = make_float2(0.f, 0.f);
                uint32_t pk[16];
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    const float2 xa = __ffma2_rn(make_float2(f(4 * u), f(4 * u + 1)), sc2, nma2);
                    const float2 xb = __ffma2_rn(make_float2(f(4 * u + 2), f(4 * u + 3)), sc2, nmb2);
                    const float2 ea = make_float2(ex2(xa.x), ex2(xa.y)), eb = make_float2(ex2(xb.x), ex2(xb.y));
                    lsa = __fadd2_rn(lsa, ea);
                    lsb = __fadd2_rn(lsb, eb);
                    __nv_bfloat162 ha = __floats2bfloat162_rn(ea.x, ea.y), hb = __floats2bfloat162_rn(eb.x, eb.y);
                    pk[2 * u] = *reinterpret_cast<uint32_t *>(&ha);
                    pk[2 * u + 1] = *reinterpret_cast<uint32_t *>(&hb);
                }
                l_a += lsa.x + lsa.y;
                l_b += lsb.x + lsb.y;

                if (raise && !first) {
                    // O may only be rescaled once the previous value product is complete
                    wait(bar(&bars->pv_done[(it - 1) & 1]), ((it - 1) >> 1) & 1, abort_s, p.error_flag);
                    tc_fence_after();
#pragma unroll 1
                    for (int c = 0; c < D; c += 64) {
                        uint32_t o[32];
                        tmem_ld_16x256b_x8(tmem + lane_base + kTmemO + c, o);
                        tmem_wait_ld();
#pragma unroll
                        for (int u = 0; u < 8; ++u) {
                            o[4 * u + 0] = __float_as_uint(__uint_as_float(o[4 * u + 0]) * alpha_a);
                            o[4 * u + 1] = __float_as_uint(__uint_as_float(o[4 * u + 1]) * alpha_a);
                            o[4 * u + 2] = __float_as_uint(__uint_as_float(o[4 * u + 2]) * alpha_b);
                            o[4 * u + 3] = __float_as_uint(__uint_as_float(o[4 * u + 3]) * alpha_b);
                        }
                        tmem_st_16x256b_x8(tmem + lane_base + kTmemO + c, o);
                    }
                    tmem_wait_st();
                }
                // P (bf16 pairs) goes to probability tile it & 1, which the value product of tile it-2 has read by
                // now; the pair of keys 8u + 2 cpair, + 1 is 32-bit column 4u + cpair
                if (it >= 2) {
                    wait(bar(&bars->pv_done[buf]), ((it - 2) >> 1) & 1, abort_s, p.error_flag);
                    tc_fence_after();
                }
                tmem_st_16x128b_x8(tmem + lane_base + kTmemP + buf * 32, pk);
                tmem_wait_st();
                // one barrier per probability tile: a warp may be a tile ahead of a slower one (never two: the
                // store above waits for the value product of tile it-2, which needs every warp's P[it-2])
                tc_fence_before();
                mbar_arrive(bar(&bars->p_full[buf]));
            }

            // ---- segment epilogue
            // The last value product (products complete in issue order, so the others are done too).
            // A parity wait can only tell a barrier's current phase from the one before it, which is
            // why the completions alternate between two barriers: when a thread waits for product i on
            // barrier i & 1, product i-2 is complete (the scores of tile i existed) and product i+2
            // cannot have been issued (it needs this thread's P), so the barrier is at most one phase
            // ahead of the waiter.  With a single barrier a thread arriving here after BOTH of the last
            // two products had completed saw the parity it was waiting to change and slept until the
            // watchdog woke it, about once in a thousand calls.
            wait(bar(&bars->pv_done[(it - 1) & 1]), ((it - 1) >> 1) & 1, abort_s, p.error_flag);
            tc_fence_after();
            // the row sums: the four shares of the quad
            l_a += __shfl_xor_sync(0xffffffffu, l_a, 1);
            l_b += __shfl_xor_sync(0xffffffffu, l_b, 1);
            l_a += __shfl_xor_sync(0xffffffffu, l_a, 2);
            l_b += __shfl_xor_sync(0xffffffffu, l_b, 2);
            if (sg.full) {
                const float inv_a = 1.f / l_a, inv_b = 1.f / l_b;   // l > 0 on a valid row: every node sees itself
                __nv_bfloat16 *dst_a = p.out + (((size_t)sg.b * p.T + j_a) * p.Hq + hq_a) * D + 2 * cpair;
                __nv_bfloat16 *dst_b = p.out + (((size_t)sg.b * p.T + j_b) * p.Hq + hq_b) * D + 2 * cpair;
#pragma unroll 1
                for (int c = 0; c < D; c += 64) {
                    uint32_t o[32];
                    tmem_ld_16x256b_x8(tmem + lane_base + kTmemO + c, o);
                    tmem_wait_ld();
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        if (ok_a)
                            *reinterpret_cast<__nv_bfloat162 *>(dst_a + c + 8 * u) =
                                __floats2bfloat162_rn(__uint_as_float(o[4 * u]) * inv_a, __uint_as_float(o[4 * u + 1]) * inv_a);
                        if (ok_b)
                            *reinterpret_cast<__nv_bfloat162 *>(dst_b + c + 8 * u) =
                                __floats2bfloat162_rn(__uint_as_float(o[4 * u + 2]) * inv_b, __uint_as_float(o[4 * u + 3]) * inv_b);
                    }
                }
                if (p.lse && cpair == 0) {
                    if (ok_a) p.lse[((size_t)sg.b * p.T + j_a) * p.Hq + hq_a] = (m_a + log2f(l_a)) * 0.6931471805599453f;
                    if (ok_b) p.lse[((size_t)sg.b * p.T + j_b) * p.Hq + hq_b] = (m_b + log2f(l_b)) * 0.6931471805599453f;
                }
            } else {
                // (single-launch kernel: slot = this CTA; the cluster's CTAs fetch the rows they merge from there)
                float *po_a = p.partial_o + ((size_t)sg.slot * kTileM + row_a) * D + 2 * cpair;
                float *po_b = p.partial_o + ((size_t)sg.slot * kTileM + row_b) * D + 2 * cpair;
#pragma unroll 1
                for (int c = 0; c < D; c += 64) {
                    uint32_t o[32];
                    tmem_ld_16x256b_x8(tmem + lane_base + kTmemO + c, o);
                    tmem_wait_ld();
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        *reinterpret_cast<uint2 *>(po_a + c + 8 * u) = make_uint2(o[4 * u], o[4 * u + 1]);
                        *reinterpret_cast<uint2 *>(po_b + c + 8 * u) = make_uint2(o[4 * u + 2], o[4 * u + 3]);
                    }
                }
                if (cpair == 0) {
                    *reinterpret_cast<float2 *>(p.partial_ml + ((size_t)sg.slot * kTileM + row_a) * 2) = make_float2(m_a, l_a);
                    *reinterpret_cast<float2 *>(p.partial_ml + ((size_t)sg.slot * kTileM + row_b) * 2) = make_float2(m_b, l_b);
                }
            }
            tc_fence_before();
        }
    }

    tc_fence_before();
    __syncthreads();
    if constexpr (kSmall) {
        // The shares of a unit meet here: CTA r of the cluster merges its r-th part of the unit's rows out of
        // every CTA's partial (m* = max m_s, l* = sum l_s 2^(m_s - m*), O = sum O_s 2^(m_s - m*) / l*)
        // and writes them.  A rejected sequence, or a CTA that gave up on a bounded wait, gets zero rows.
        const bool multi = cl_size > 1;
        const int rb = bars->reject;   // complete: every warp has passed the barrier above
        reject = (rb & 8) ? *p.error_flag : (rb & 1) ? READER_ERR_BAD_TREE : (rb & 2) ? READER_ERR_CAPACITY : (rb & 4) ? READER_ERR_BAD_PAGE : 0;
        if (tid == 0 && cl_rank == 0 && mine.h == 0 && mine.mt == 0) p.status[mine.b] = reject;
        const bool gave_up = *abort_s != 0;
        if (multi) {
            if (tid == 0) p.split_desc[cta].b = gave_up ? 1 : 0;   // this CTA's give-up flag, beside its partial
            cluster_arrive_release();
            cluster_wait_acquire();
        }
        if (warp < kSoftmaxWarps && (multi || reject != 0 || gave_up)) {
            // the unit's real rows (a small tree fills only the first of the 128) are dealt out evenly
            const int rows_real = min(kTileM, p.T * p.G - mine.mt * kTileM);
            const int rows_per = (rows_real + (int)cl_size - 1) / (int)cl_size;
            const bool has_cols = lane * 4 < D;
            const int cta0 = cta - (int)cl_rank;   // the cluster's first CTA: share q lies in partial slot cta0 + q
            int peer_flag = 0;   // consumed after the first row's loads have been issued: one round trip to L2, not two
            if (multi && lane < (int)cl_size) peer_flag = __ldcg(&p.split_desc[cta0 + lane].b);
            bool peer_gave_up = false, flags_read = false;
            for (int rr = warp; rr < rows_per; rr += kSoftmaxWarps) {
                const int row = (int)cl_rank * rows_per + rr;
                const int grow = mine.mt * kTileM + row;
                if (row >= rows_real) continue;
                float mstar = -INFINITY, lstar = 0.f;
                float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
                bool bad = reject != 0 || gave_up;
                if (multi && reject == 0) {
                    // every share's row in flight at once.  The shares travel through the workspace (L2), not through
                    // distributed shared memory: reads of another CTA's shared memory came back one at a time,
                    // 0.3 us each, which made this merge 5 us long on eight shares.
                    constexpr int kMaxCluster = 8;
                    float2 ml[kMaxCluster];
                    float4 o[kMaxCluster];
#pragma unroll
                    for (int q = 0; q < kMaxCluster; ++q) {
                        ml[q] = make_float2(-INFINITY, 0.f);
                        o[q] = make_float4(0.f, 0.f, 0.f, 0.f);
                        if (q < (int)cl_size) {
                            ml[q] = __ldcg(reinterpret_cast<const float2 *>(p.partial_ml + ((size_t)(cta0 + q) * kTileM + row) * 2));
                            if (has_cols) o[q] = __ldcg(reinterpret_cast<const float4 *>(p.partial_o + ((size_t)(cta0 + q) * kTileM + row) * D + lane * 4));
                        }
                    }
#pragma unroll
                    for (int q = 0; q < kMaxCluster; ++q) mstar = fmaxf(mstar, ml[q].x);
                    if (!flags_read) {
                        peer_gave_up = __any_sync(0xffffffffu, peer_flag != 0);
                        flags_read = true;
                    }
                    bad = bad || peer_gave_up;
#pragma unroll
                    for (int q = 0; q < kMaxCluster; ++q) {
                        const float wgt = ml[q].x == -INFINITY ? 0.f : exp2f(ml[q].x - mstar);   // an empty share holds no row
                        lstar = fmaf(ml[q].y, wgt, lstar);
                        acc.x = fmaf(wgt == 0.f ? 0.f : o[q].x, wgt, acc.x);
                        acc.y = fmaf(wgt == 0.f ? 0.f : o[q].y, wgt, acc.y);
                        acc.z = fmaf(wgt == 0.f ? 0.f : o[q].z, wgt, acc.z);
                        acc.w = fmaf(wgt == 0.f ? 0.f : o[q].w, wgt, acc.w);
                    }
                }
                const int j = grow / p.G, hq = mine.h * p.G + grow % p.G;
                const size_t orow = ((size_t)mine.b * p.T + j) * p.Hq + hq;
                const float inv = bad ? 0.f : 1.f / lstar;
                if (has_cols) {
                    __nv_bfloat162 lo = __floats2bfloat162_rn(bad ? 0.f : acc.x * inv, bad ? 0.f : acc.y * inv);
                    __nv_bfloat162 hi = __floats2bfloat162_rn(bad ? 0.f : acc.z * inv, bad ? 0.f : acc.w * inv);
                    uint2 v;
                    v.x = *reinterpret_cast<uint32_t *>(&lo);
                    v.y = *reinterpret_cast<uint32_t *>(&hi);
                    *reinterpret_cast<uint2 *>(p.out + orow * D + lane * 4) = v;
                }
                if (p.lse && lane == 0) p.lse[orow] = bad ? 0.f : (mstar + log2f(lstar)) * 0.6931471805599453f;
                if (bad && reject == 0 && lane == 0) atomicMax(&p.status[mine.b], (int32_t)READER_ERR_TIMEOUT);
            }
        }
    }
    if (warp == kMmaWarp) {
        tc_fence_after();
        tmem_dealloc(tmem, kTmemCols);
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// 2-D view of a pool (or of a padded batch cache): all its rows of head_dim columns; box = 64 x 64.
bool encode_pool_map(void *fn, CUtensorMap *map, const void *pool, int64_t rows, int D) {
    const cuuint64_t dims[2] = {(cuuint64_t)D, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)D * 2};
    const cuuint32_t box[2] = {64, (cuuint32_t)kPage};
    const cuuint32_t estr[2] = {1, 1};
    return reinterpret_cast<EncodeTiledFn>(fn)(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(pool), dims,
                                               strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// 3-D view of a tree tensor [B*T nodes][Hkv][D]: box = 64 columns x 1 head x 64 nodes.
bool encode_tree_map(void *fn, CUtensorMap *map, const void *tree, int64_t nodes, int Hkv, int D) {
    const cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)Hkv, (cuuint64_t)nodes};
    const cuuint64_t strides[2] = {(cuuint64_t)D * 2, (cuuint64_t)Hkv * D * 2};
    const cuuint32_t box[3] = {64, 1, (cuuint32_t)kPage};
    const cuuint32_t estr[3] = {1, 1, 1};
    return reinterpret_cast<EncodeTiledFn>(fn)(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(tree), dims,
                                               strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// 4-D view of q [B][T][Hq][D]: box = 64 columns x G heads x 128/G nodes x 1 sequence, which lands in
// shared memory as 128 rows ordered (node, group member).
bool encode_q_map(void *fn, CUtensorMap *map, const void *q, int B, int T, int Hq, int G, int D) {
    const cuuint64_t dims[4] = {(cuuint64_t)D, (cuuint64_t)Hq, (cuuint64_t)T, (cuuint64_t)B};
    const cuuint64_t strides[3] = {(cuuint64_t)D * 2, (cuuint64_t)Hq * D * 2, (cuuint64_t)T * Hq * D * 2};
    const cuuint32_t box[4] = {64, (cuuint32_t)G, (cuuint32_t)(kTileM / G), 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    return reinterpret_cast<EncodeTiledFn>(fn)(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(q), dims,
                                               strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

// Cached TMA descriptors.  A model calls the kernel once per layer and step with that layer's pools, so
// the pool descriptors are kept for the last kPoolEntries distinct pools (round robin); the tree and query
// tensors change with every call in a real decode loop and get one entry each.
constexpr int kPoolEntries = 128;
struct PoolMaps {
    const void *k_pool = nullptr, *v_pool = nullptr;
    int64_t rows = -1;
    int D = 0;
    alignas(64) CUtensorMap kmap, vmap;
};
struct Sm100Maps {
    PoolMaps pools[kPoolEntries];
    int next_pool = 0;
    const void *k_tree = nullptr, *v_tree = nullptr;
    int64_t nodes = -1;
    int tree_heads = 0, tree_D = 0;
    const void *q = nullptr;
    int qB = -1, qT = 0, qHq = 0, qG = 0, qD = 0;
    alignas(64) CUtensorMap ktmap, vtmap, qmap;
};

// The tensor-core kernel is the library's attention path: a device on which it cannot run (no
// cuTensorMapEncodeTiled in the driver, too little opt-in shared memory) is refused here, so that no call
// is ever served silently by the CUDA-core kernel.
reader_status sm100_host_init(Sm100Host *h, int device) {
    h->encode_tiled = nullptr;
    h->smem_optin = 0;
    h->ready = false;
    h->attr_set = false;
    h->maps = nullptr;
    void *fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess || !fn) {
        cudaGetLastError();
        return READER_ERR_UNSUPPORTED;
    }
    if (cudaDeviceGetAttribute(&h->smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, device) != cudaSuccess) {
        cudaGetLastError();
        return READER_ERR_CUDA;
    }
    if (h->smem_optin < Cfg<128>::kSmemBytes) return READER_ERR_UNSUPPORTED;
    h->maps = new (std::nothrow) Sm100Maps();
    if (!h->maps) return READER_ERR_CUDA;
    h->encode_tiled = fn;
    h->ready = true;
    return READER_OK;
}

void sm100_host_destroy(Sm100Host *h) {
    delete h->maps;
    h->maps = nullptr;
    h->ready = false;
}

bool sm100_supports(const Sm100Host *h, const AttnParams &p, float softmax_scale) {
    if (!h->ready) return false;
    if (!(softmax_scale > 0.f) || softmax_scale > 3.0e38f) return false;   // the row maximum is taken before scaling
    const int64_t rows = p.pool_rows;
    if (p.G > kTileM || kTileM % p.G != 0) return false;   // a query tile is a box of whole nodes
    return (p.D == 64 || p.D == 128) && rows >= 1 && rows < ((int64_t)1 << 31);
}

// small_cluster = 0: the general kernel on the schedule the preparation kernel left in the workspace;
// 1, 2, 4 or 8: the single-launch kernel, one cluster of that many CTAs per (sequence, KV head, M tile).
reader_status launch_attn_sm100(Sm100Host *h, const AttnParams &p, int small_cluster, cudaStream_t st) {
    if (!h->attr_set) {
        if (cudaFuncSetAttribute(attn_sm100_kernel<128, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<128>::kSmemBytes) != cudaSuccess ||
            cudaFuncSetAttribute(attn_sm100_kernel<64, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<64>::kSmemBytes) != cudaSuccess ||
            cudaFuncSetAttribute(attn_sm100_kernel<128, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<128>::kSmemBytes) != cudaSuccess ||
            cudaFuncSetAttribute(attn_sm100_kernel<64, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<64>::kSmemBytes) != cudaSuccess ||
            cudaFuncSetAttribute(attn_sm100_kernel<128, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<128>::kSmemBytesSmall) != cudaSuccess ||
            cudaFuncSetAttribute(attn_sm100_kernel<64, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<64>::kSmemBytesSmall) != cudaSuccess) {
            cudaGetLastError();
            return READER_ERR_CUDA;
        }
        h->attr_set = true;
    }
    Sm100Maps *m = h->maps;
    const int64_t rows = p.pool_rows;
    PoolMaps *pm = nullptr;
    for (int i = 0; i < kPoolEntries && !pm; ++i) {
        PoolMaps &e = m->pools[i];
        if (e.k_pool == p.k_pool && e.v_pool == p.v_pool && e.rows == rows && e.D == p.D) pm = &e;
    }
    if (!pm) {
        pm = &m->pools[m->next_pool];
        m->next_pool = (m->next_pool + 1) % kPoolEntries;
        pm->rows = -1;
        if (!encode_pool_map(h->encode_tiled, &pm->kmap, p.k_pool, rows, p.D) ||
            !encode_pool_map(h->encode_tiled, &pm->vmap, p.v_pool, rows, p.D))
            return READER_ERR_CUDA;
        pm->k_pool = p.k_pool; pm->v_pool = p.v_pool; pm->rows = rows; pm->D = p.D;
    }
    const int64_t nodes = (int64_t)p.B * p.T;
    if (m->k_tree != p.k_tree || m->v_tree != p.v_tree || m->nodes != nodes || m->tree_heads != p.Hkv || m->tree_D != p.D) {
        if (!encode_tree_map(h->encode_tiled, &m->ktmap, p.k_tree, nodes, p.Hkv, p.D) ||
            !encode_tree_map(h->encode_tiled, &m->vtmap, p.v_tree, nodes, p.Hkv, p.D)) {
            m->nodes = -1;
            return READER_ERR_CUDA;
        }
        m->k_tree = p.k_tree; m->v_tree = p.v_tree; m->nodes = nodes; m->tree_heads = p.Hkv; m->tree_D = p.D;
    }
    if (m->q != p.q || m->qB != p.B || m->qT != p.T || m->qHq != p.Hq || m->qG != p.G || m->qD != p.D) {
        if (!encode_q_map(h->encode_tiled, &m->qmap, p.q, p.B, p.T, p.Hq, p.G, p.D)) {
            m->qB = -1;
            return READER_ERR_CUDA;
        }
        m->q = p.q; m->qB = p.B; m->qT = p.T; m->qHq = p.Hq; m->qG = p.G; m->qD = p.D;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(kThreads);
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // prologue overlaps the kernel before it
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    auto kernel = p.D == 128 ? (p.valid_bits ? attn_sm100_kernel<128, true, false> : attn_sm100_kernel<128, false, false>)
                             : (p.valid_bits ? attn_sm100_kernel<64, true, false> : attn_sm100_kernel<64, false, false>);
    if (small_cluster > 0) {
        if (p.valid_bits) return READER_ERR_UNSUPPORTED;
        const int n_mtiles = (p.T * p.G + kTileM - 1) / kTileM;
        cfg.gridDim = dim3((unsigned)(p.B * p.Hkv * n_mtiles * small_cluster));
        cfg.dynamicSmemBytes = p.D == 128 ? Cfg<128>::kSmemBytesSmall : Cfg<64>::kSmemBytesSmall;
        kernel = p.D == 128 ? attn_sm100_kernel<128, false, true> : attn_sm100_kernel<64, false, true>;
        if (small_cluster > 1) {
            attr[1].id = cudaLaunchAttributeClusterDimension;
            attr[1].val.clusterDim.x = (unsigned)small_cluster;
            attr[1].val.clusterDim.y = 1;
            attr[1].val.clusterDim.z = 1;
            cfg.numAttrs = 2;
        }
    } else {
        cfg.gridDim = dim3(p.sched.n_ctas);
        cfg.dynamicSmemBytes = p.D == 128 ? Cfg<128>::kSmemBytes : Cfg<64>::kSmemBytes;
    }
    const cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, p, pm->kmap, pm->vmap, m->ktmap, m->vtmap, m->qmap);
    if (e != cudaSuccess) {
        cudaGetLastError();
        return READER_ERR_CUDA;
    }
    return READER_OK;
}

}  // namespace reader
