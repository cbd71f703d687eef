// Tree-masked verify attention (Sec. 3.2) on the sm_100a tensor cores.
//
// Two persistent CTAs per SM each walk their range of the flattened split-KV tile list.  For every unit
// (sequence, KV head, 128 query rows) it computes S = Q K^T and O += P V with tcgen05.mma, one KV
// tile of 64 keys (one cache page, or 64 tree nodes) at a time:
//
//   warp 4      producer: full cache pages arrive by TMA (two 64x64 boxes per K and per V tile,
//               128-byte swizzle) into a ring of kStages stages; the ragged last page and the
//               tree tiles are copied with ordinary loads and zero-filled past their end, so that
//               bytes beyond a sequence's length can never reach a product
//   warp 5      MMA issuer: S[t+1] = Q K[t+1]^T is issued ahead of O += P[t] V[t], so the tensor
//               pipe works on the next scores while the softmax warps are busy with this tile
//   warps 0-3   softmax: thread r owns query row r = TMEM lane r.  Scores come from TMEM, the
//               ancestor bitmask / length mask is applied, the running maximum is raised only
//               when it grows by more than 2^8 (the accumulator in TMEM is rescaled then),
//               probabilities go to shared memory as the bf16 A operand of the value product.
//               The same threads stage Q at the start of a segment and write O (or an (m, l, O)
//               partial) at its end.
//
// TMEM: columns 0-127 hold two score buffers of 64 columns, columns 128.. hold O (head_dim
// columns), all fp32, lane = query row.  Every wait on an mbarrier is bounded: after one second a
// CTA raises the error flag in the workspace, stops waiting and runs to its end.
#include <cuda.h>

#include <new>

#include "ptx_sm100.cuh"
#include "verify_attn_sm100.cuh"

namespace reader {
namespace {

using namespace ptx;

constexpr int kStages = 2;          // per CTA; two CTAs share an SM, so four tiles are in flight per SM
constexpr int kThreads = 192;
constexpr int kProducerWarp = 4;
constexpr int kMmaWarp = 5;
constexpr uint64_t kWaitLimitNs = 1000000000ull;
constexpr float kRaiseMaxBy = 8.f;   // log2 units
constexpr uint32_t kTmemCols = 256;
constexpr uint32_t kTmemO = 128;

template <int D>
struct Cfg {
    static constexpr int kHalves = D / 64;                 // 64-column (128-byte) blocks per row
    static constexpr int kHalfRowsQ = kTileM * 128;        // bytes of one 64-column block of Q
    static constexpr int kHalfRowsKV = kPage * 128;        // bytes of one 64-column block of a KV tile
    static constexpr int kQBytes = kTileM * D * 2;
    static constexpr int kPBytes = kTileM * kPage * 2;
    static constexpr int kTileBytes = kPage * D * 2;
    static constexpr int kStageBytes = 2 * kTileBytes;
    static constexpr int kOffQ = 0;
    static constexpr int kOffP = kQBytes;
    static constexpr int kOffStages = kOffP + kPBytes;
    static constexpr int kOffBars = kOffStages + kStages * kStageBytes;
    static constexpr int kSmemBytes = kOffBars + 256;   // + barriers; two CTAs of head_dim 128 fit one SM
};

struct Bars {
    uint64_t kv_full[kStages], kv_empty[kStages];
    uint64_t q_full, s_full[2], s_empty[2], p_full, pv_done;
    uint32_t tmem_base;
    int32_t abort;
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

template <int D>
__global__ void __launch_bounds__(kThreads, 2)
attn_sm100_kernel(const AttnParams p, const __grid_constant__ CUtensorMap kmap, const __grid_constant__ CUtensorMap vmap) {
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

    const uint32_t sQ = base + C::kOffQ, sP = base + C::kOffP, sStages = base + C::kOffStages;
    auto bar = [&](const uint64_t *b) { return smem_u32(b); };

    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(bar(&bars->kv_full[s]), 1);
            mbar_init(bar(&bars->kv_empty[s]), 1);
        }
        mbar_init(bar(&bars->q_full), kTileM);
        for (int s = 0; s < 2; ++s) {
            mbar_init(bar(&bars->s_full[s]), 1);
            mbar_init(bar(&bars->s_empty[s]), kTileM);
        }
        mbar_init(bar(&bars->p_full), kTileM);
        mbar_init(bar(&bars->pv_done), 1);
        bars->abort = 0;
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

    const int W = p.sched.seq_tile_start[p.B];
    const int w_begin = range_begin(cta, p.sched.n_ctas, W);
    const int w_end = range_begin(cta + 1, p.sched.n_ctas, W);

    if (warp == kProducerWarp) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            prefetch_tensormap(&kmap);
            prefetch_tensormap(&vmap);
        }
        int it = 0;
        int w = w_begin;
        while (w < w_end) {
            const Segment sg = segment_at(p.sched, p.B, cta, w, w_end);
            w += sg.tile_end - sg.tile_begin;
            const int L = p.seq_lens[sg.b];
            for (int t0 = sg.tile_begin; t0 < sg.tile_end; t0 += 32) {
                const int tt = t0 + lane;
                const int my_page = (tt < sg.tile_end && tt < sg.npages) ? p.page_table[(size_t)sg.b * p.max_pages + tt] : 0;
                const int n = min(32, sg.tile_end - t0);
                for (int i = 0; i < n; ++i, ++it) {
                    const int t = t0 + i;
                    const int page = __shfl_sync(0xffffffffu, my_page, i);
                    const int stage = it % kStages;
                    wait(bar(&bars->kv_empty[stage]), ((it / kStages) & 1) ^ 1, abort_s, p.error_flag);
                    const uint32_t kdst = sStages + stage * C::kStageBytes, vdst = kdst + C::kTileBytes;
                    const uint32_t full = bar(&bars->kv_full[stage]);
                    const bool whole_page = t < sg.npages && L - t * kPage >= kPage;
                    if (whole_page) {
                        if (lane == 0) {
                            mbar_arrive_expect_tx(full, C::kStageBytes);
                            const int row = (page * p.Hkv + sg.h) * kPage;
#pragma unroll
                            for (int hf = 0; hf < C::kHalves; ++hf) {
                                tma_load_2d(kdst + hf * C::kHalfRowsKV, &kmap, full, hf * 64, row);
                                tma_load_2d(vdst + hf * C::kHalfRowsKV, &vmap, full, hf * 64, row);
                            }
                        }
                    } else {
                        const __nv_bfloat16 *ksrc, *vsrc;
                        size_t stride;
                        int valid;
                        if (t < sg.npages) {
                            const size_t at = ((size_t)page * p.Hkv + sg.h) * kPage * D;
                            ksrc = p.k_pool + at; vsrc = p.v_pool + at;
                            stride = D;
                            valid = L - t * kPage;
                        } else {
                            const int kt = t - sg.npages;
                            const size_t at = (((size_t)sg.b * p.T + kt * kPage) * p.Hkv + sg.h) * D;
                            ksrc = p.k_tree + at; vsrc = p.v_tree + at;
                            stride = (size_t)p.Hkv * D;
                            valid = min(kPage, p.T - kt * kPage);
                        }
                        constexpr int kChunks = D / 8;
#pragma unroll 4
                        for (int c = lane; c < kPage * kChunks; c += 32) {
                            const int rr = c / kChunks, cc = c % kChunks;
                            uint4 kv = make_uint4(0, 0, 0, 0), vv = make_uint4(0, 0, 0, 0);
                            if (rr < valid) {
                                kv = *reinterpret_cast<const uint4 *>(ksrc + rr * stride + cc * 8);
                                vv = *reinterpret_cast<const uint4 *>(vsrc + rr * stride + cc * 8);
                            }
                            const uint32_t off = (cc >> 3) * C::kHalfRowsKV + rr * 128 + (((cc & 7) ^ (rr & 7)) << 4);
                            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(kdst + off), "r"(kv.x), "r"(kv.y), "r"(kv.z), "r"(kv.w) : "memory");
                            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(vdst + off), "r"(vv.x), "r"(vv.y), "r"(vv.z), "r"(vv.w) : "memory");
                        }
                        fence_proxy_async();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(full);
                    }
                }
            }
        }
        // a CTA that gave up must not exit under its own copies: let the last ones land (bounded)
        if (*abort_s) {
            const uint64_t t0 = globaltimer_ns();
            for (int i = max(0, it - kStages); i < it; ++i)
                while (!mbar_try_wait(bar(&bars->kv_full[i % kStages]), (i / kStages) & 1) &&
                       globaltimer_ns() - t0 < 20000000ull) {
                }
        }
    } else if (warp == kMmaWarp) {
        // ------------------------------------------------------------------ MMA issuer
        constexpr uint32_t kIdescQK = idesc_bf16_f32(kTileM, kPage, false, false);
        constexpr uint32_t kIdescPV = idesc_bf16_f32(kTileM, D, false, true);
        auto issue_qk = [&](int i) {
            const int stage = i % kStages, buf = i & 1;
            wait(bar(&bars->kv_full[stage]), (i / kStages) & 1, abort_s, p.error_flag);
            wait(bar(&bars->s_empty[buf]), ((i >> 1) & 1) ^ 1, abort_s, p.error_flag);
            tc_fence_after();
            if (lane == 0) {
                const uint32_t kbase = sStages + stage * C::kStageBytes;
#pragma unroll
                for (int hf = 0; hf < C::kHalves; ++hf)
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk) {
                        const uint64_t a = smem_desc_sw128(sQ + hf * C::kHalfRowsQ + kk * 32, 16, 1024);
                        const uint64_t b = smem_desc_sw128(kbase + hf * C::kHalfRowsKV + kk * 32, 16, 1024);
                        mma_bf16_ss(tmem + buf * kPage, a, b, kIdescQK, (hf | kk) != 0);
                    }
                mma_commit(bar(&bars->s_full[buf]));
            }
            __syncwarp();
        };
        int it = 0, seg = 0;
        int w = w_begin;
        while (w < w_end) {
            const Segment sg = segment_at(p.sched, p.B, cta, w, w_end);
            const int n = sg.tile_end - sg.tile_begin;
            w += n;
            wait(bar(&bars->q_full), seg & 1, abort_s, p.error_flag);
            tc_fence_after();
            issue_qk(it);
            for (int t = 0; t < n; ++t) {
                if (t + 1 < n) issue_qk(it + t + 1);
                wait(bar(&bars->p_full), (it + t) & 1, abort_s, p.error_flag);
                tc_fence_after();
                if (lane == 0) {
                    const int stage = (it + t) % kStages;
                    const uint32_t vbase = sStages + stage * C::kStageBytes + C::kTileBytes;
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk) {
                        const uint64_t a = smem_desc_sw128(sP + kk * 32, 16, 1024);
                        const uint64_t b = smem_desc_sw128(vbase + kk * 2048, C::kHalfRowsKV, 1024);
                        mma_bf16_ss(tmem + kTmemO, a, b, kIdescPV, (t | kk) != 0);
                    }
                    mma_commit(bar(&bars->kv_empty[stage]));
                    mma_commit(bar(&bars->pv_done));
                }
                __syncwarp();
            }
            it += n;
            ++seg;
        }
    } else {
        // ------------------------------------------------------------------ softmax / epilogue
        const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
        int it = 0;
        int w = w_begin;
        while (w < w_end) {
            const Segment sg = segment_at(p.sched, p.B, cta, w, w_end);
            w += sg.tile_end - sg.tile_begin;
            const int L = p.seq_lens[sg.b];
            const int grow = sg.mt * kTileM + tid;
            const bool row_ok = grow < p.T * p.G;
            const int j = row_ok ? grow / p.G : 0;
            const int hq = sg.h * p.G + (row_ok ? grow % p.G : 0);
            const size_t qrow = (((size_t)sg.b * p.T + j) * p.Hq + hq) * D;

            // stage this thread's query row (128-byte swizzle, zero for padding rows)
            {
                const uint4 *src = reinterpret_cast<const uint4 *>(p.q + qrow);
#pragma unroll
                for (int c = 0; c < D / 8; ++c) {
                    const uint4 v = row_ok ? src[c] : make_uint4(0, 0, 0, 0);
                    const uint32_t off = (c >> 3) * C::kHalfRowsQ + tid * 128 + (((c & 7) ^ (tid & 7)) << 4);
                    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(sQ + off), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
                }
                fence_proxy_async();
                mbar_arrive(bar(&bars->q_full));
            }
            uint64_t anc_lo = 0, anc_hi = 0;
            if (row_ok) {
                anc_lo = p.anc[((size_t)sg.b * p.T + j) * 2 + 0];
                anc_hi = p.anc[((size_t)sg.b * p.T + j) * 2 + 1];
            }

            float m_used = -INFINITY, l = 0.f;
            for (int t = sg.tile_begin; t < sg.tile_end; ++t, ++it) {
                uint64_t vis;
                if (t < sg.npages) {
                    const int valid = L - t * kPage;
                    vis = valid >= kPage ? ~0ull : ((1ull << valid) - 1);
                } else {
                    vis = (t - sg.npages) == 0 ? anc_lo : anc_hi;
                }
                const int buf = it & 1;
                wait(bar(&bars->s_full[buf]), (it >> 1) & 1, abort_s, p.error_flag);
                tc_fence_after();
                uint32_t s0[32], s1[32];
                tmem_ld32(tmem + lane_base + buf * kPage, s0);
                tmem_ld32(tmem + lane_base + buf * kPage + 32, s1);
                tmem_wait_ld();
                tc_fence_before();
                mbar_arrive(bar(&bars->s_empty[buf]));

                if (vis != ~0ull) {
                    const uint32_t lo = (uint32_t)vis, hi = (uint32_t)(vis >> 32);
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        if (!((lo >> i) & 1u)) s0[i] = 0xff800000u;
                        if (!((hi >> i) & 1u)) s1[i] = 0xff800000u;
                    }
                }
                float mxs[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) mxs[i] = fmaxf(__uint_as_float(s0[i]), __uint_as_float(s1[i]));
#pragma unroll
                for (int i = 8; i < 32; ++i) mxs[i & 7] = fmaxf(mxs[i & 7], fmaxf(__uint_as_float(s0[i]), __uint_as_float(s1[i])));
                const float mx = fmaxf(fmaxf(fmaxf(mxs[0], mxs[1]), fmaxf(mxs[2], mxs[3])),
                                       fmaxf(fmaxf(mxs[4], mxs[5]), fmaxf(mxs[6], mxs[7])));
                const float m_new = fmaxf(m_used, mx * p.scale_log2);
                const bool first = t == sg.tile_begin;
                const bool raise = __any_sync(0xffffffffu, m_new > m_used + kRaiseMaxBy);
                float alpha = 1.f;
                if (raise || first) {
                    alpha = (m_new == -INFINITY) ? 1.f : ex2(m_used - m_new);
                    m_used = m_new;
                    l *= alpha;
                }
                const float neg_m = (m_used == -INFINITY) ? 0.f : -m_used;
                float ls[4] = {0.f, 0.f, 0.f, 0.f};
                uint32_t pk[32];
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const float a = ex2(fmaf(__uint_as_float(s0[2 * i]), p.scale_log2, neg_m));
                    const float b = ex2(fmaf(__uint_as_float(s0[2 * i + 1]), p.scale_log2, neg_m));
                    ls[i & 3] += a + b;
                    __nv_bfloat162 h2 = __floats2bfloat162_rn(a, b);
                    pk[i] = *reinterpret_cast<uint32_t *>(&h2);
                }
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const float a = ex2(fmaf(__uint_as_float(s1[2 * i]), p.scale_log2, neg_m));
                    const float b = ex2(fmaf(__uint_as_float(s1[2 * i + 1]), p.scale_log2, neg_m));
                    ls[i & 3] += a + b;
                    __nv_bfloat162 h2 = __floats2bfloat162_rn(a, b);
                    pk[16 + i] = *reinterpret_cast<uint32_t *>(&h2);
                }
                l += (ls[0] + ls[1]) + (ls[2] + ls[3]);

                // the previous value product must be complete before P or O are touched
                if (it > 0) {
                    wait(bar(&bars->pv_done), (it - 1) & 1, abort_s, p.error_flag);
                    tc_fence_after();
                }
                if (raise && !first) {
#pragma unroll 1
                    for (int c = 0; c < D; c += 32) {
                        uint32_t o[32];
                        tmem_ld32(tmem + lane_base + kTmemO + c, o);
                        tmem_wait_ld();
#pragma unroll
                        for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
                        tmem_st32(tmem + lane_base + kTmemO + c, o);
                    }
                    tmem_wait_st();
                }
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    const uint32_t off = tid * 128 + ((c ^ (tid & 7)) << 4);
                    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(sP + off), "r"(pk[4 * c]), "r"(pk[4 * c + 1]), "r"(pk[4 * c + 2]), "r"(pk[4 * c + 3]) : "memory");
                }
                fence_proxy_async();
                tc_fence_before();
                mbar_arrive(bar(&bars->p_full));
            }

            // ---- segment epilogue
            wait(bar(&bars->pv_done), (it - 1) & 1, abort_s, p.error_flag);
            tc_fence_after();
            if (sg.full) {
                const float inv = 1.f / l;   // l > 0 on a valid row: every node sees itself
                __nv_bfloat16 *dst = p.out + qrow;
#pragma unroll 1
                for (int c = 0; c < D; c += 32) {
                    uint32_t o[32];
                    tmem_ld32(tmem + lane_base + kTmemO + c, o);
                    tmem_wait_ld();
                    if (row_ok) {
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            uint4 v;
                            __nv_bfloat162 h0 = __floats2bfloat162_rn(__uint_as_float(o[8 * i + 0]) * inv, __uint_as_float(o[8 * i + 1]) * inv);
                            __nv_bfloat162 h1 = __floats2bfloat162_rn(__uint_as_float(o[8 * i + 2]) * inv, __uint_as_float(o[8 * i + 3]) * inv);
                            __nv_bfloat162 h2 = __floats2bfloat162_rn(__uint_as_float(o[8 * i + 4]) * inv, __uint_as_float(o[8 * i + 5]) * inv);
                            __nv_bfloat162 h3 = __floats2bfloat162_rn(__uint_as_float(o[8 * i + 6]) * inv, __uint_as_float(o[8 * i + 7]) * inv);
                            v.x = *reinterpret_cast<uint32_t *>(&h0);
                            v.y = *reinterpret_cast<uint32_t *>(&h1);
                            v.z = *reinterpret_cast<uint32_t *>(&h2);
                            v.w = *reinterpret_cast<uint32_t *>(&h3);
                            *reinterpret_cast<uint4 *>(dst + c + 8 * i) = v;
                        }
                    }
                }
                if (row_ok && p.lse)
                    p.lse[((size_t)sg.b * p.T + j) * p.Hq + hq] = (m_used + log2f(l)) * 0.6931471805599453f;
            } else {
                float *po = p.partial_o + ((size_t)sg.slot * kTileM + tid) * D;
#pragma unroll 1
                for (int c = 0; c < D; c += 32) {
                    uint32_t o[32];
                    tmem_ld32(tmem + lane_base + kTmemO + c, o);
                    tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        *reinterpret_cast<uint4 *>(po + c + 4 * i) = make_uint4(o[4 * i], o[4 * i + 1], o[4 * i + 2], o[4 * i + 3]);
                }
                *reinterpret_cast<float2 *>(p.partial_ml + ((size_t)sg.slot * kTileM + tid) * 2) = make_float2(m_used, l);
            }
            tc_fence_before();
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == kMmaWarp) {
        tc_fence_after();
        tmem_dealloc(tmem, kTmemCols);
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// 2-D view of a pool: rows = num_pages * n_kv_heads * page_size, head_dim columns; box = 64 x 64.
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

}  // namespace

struct Sm100Maps {
    const void *k_pool = nullptr, *v_pool = nullptr;
    int64_t rows = -1;
    int D = 0;
    alignas(64) CUtensorMap kmap, vmap;
};

reader_status sm100_host_init(Sm100Host *h, int device) {
    h->encode_tiled = nullptr;
    h->smem_optin = 0;
    h->ready = false;
    h->attr_set = false;
    h->maps = nullptr;
    void *fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess) {
        cudaGetLastError();
        return READER_OK;   // the CUDA-core kernel still serves every shape
    }
    if (cudaDeviceGetAttribute(&h->smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, device) != cudaSuccess) {
        cudaGetLastError();
        return READER_OK;
    }
    h->maps = new (std::nothrow) Sm100Maps();
    h->encode_tiled = fn;
    h->ready = h->maps != nullptr && h->smem_optin >= Cfg<128>::kSmemBytes;
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
    const int64_t rows = (int64_t)p.num_pages * p.Hkv * kPage;
    return (p.D == 64 || p.D == 128) && rows >= 1 && rows < ((int64_t)1 << 31);
}

reader_status launch_attn_sm100(Sm100Host *h, const AttnParams &p, const reader_kv_cache &cache, cudaStream_t st) {
    if (!h->attr_set) {
        if (cudaFuncSetAttribute(attn_sm100_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<128>::kSmemBytes) != cudaSuccess ||
            cudaFuncSetAttribute(attn_sm100_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<64>::kSmemBytes) != cudaSuccess) {
            cudaGetLastError();
            return READER_ERR_CUDA;
        }
        h->attr_set = true;
    }
    Sm100Maps *m = h->maps;
    const int64_t rows = (int64_t)cache.num_pages * cache.n_kv_heads * kPage;
    if (m->k_pool != cache.k_pool || m->v_pool != cache.v_pool || m->rows != rows || m->D != p.D) {
        if (!encode_pool_map(h->encode_tiled, &m->kmap, cache.k_pool, rows, p.D) ||
            !encode_pool_map(h->encode_tiled, &m->vmap, cache.v_pool, rows, p.D)) {
            m->rows = -1;
            return READER_ERR_CUDA;
        }
        m->k_pool = cache.k_pool; m->v_pool = cache.v_pool; m->rows = rows; m->D = p.D;
    }
    if (p.D == 128)
        attn_sm100_kernel<128><<<p.sched.n_ctas, kThreads, Cfg<128>::kSmemBytes, st>>>(p, m->kmap, m->vmap);
    else
        attn_sm100_kernel<64><<<p.sched.n_ctas, kThreads, Cfg<64>::kSmemBytes, st>>>(p, m->kmap, m->vmap);
    return READER_OK;
}

}  // namespace reader
