// Randomized decoding policy (Appendix C, "Randomized decoding"): the token the target model's
// policy emits, x* = F(P(. | prefix), U_t), by temperature sampling through the inverse CDF with
// one uniform per output position.  All nodes of one tree level propose tokens for the same
// position, so node j of sequence b uses uniforms[b][level(j) - 1].
//
// The CDF is built from integers so that no summation order can change the outcome:
//   c   = (float)(log2(e) / temperature)   (host, double division rounded once)
//   m   = row maximum (a NaN never wins; NaN in slot 0 counts as -inf)
//   x_v = (l_v - m) * c  (two fp32 roundings); NaN or x_v < -64: weight 0
//   n = rint(x_v), f = x_v - n, p = 1 + f(c1 + f(c2 + f(c3 + f(c4 + f c5)))) with fused multiply-adds,
//       c_k = ln(2)^k / k! in fp32
//   W_v = trunc(p * 2^(n + 40));  S = sum W_v;  U = trunc(u * 2^24);  thr = (S * U) >> 24
//   x*  = first v whose inclusive prefix sum of W exceeds thr (0 when S = 0)
// Top-k (top_k >= 1, 0 = off): tau = the top_k-th largest logit of the row (NaN counts as -inf); only
// logits >= tau keep their weight (ties at tau are all kept).  tau is found exactly by a radix select
// over an order-preserving 32-bit key in three passes (11 + 11 + 10 bits), restricted to the logits that
// are at least the k-th largest per-thread maximum of the max pass (an exact lower bound for k <= 256).
// Top-p (0 < top_p < 1, applied to what top-k left): with S0 the kept weight and M = max(1, (S0 *
// trunc(top_p * 2^24)) >> 24), tau_p is the largest logit t whose kept logits >= t weigh at least M;
// only logits >= tau_p stay (equal logits at the boundary are admitted together).  Found by the same
// radix select with 64-bit weight sums per bin.
// One CTA of 256 threads per row (four resident per SM; a grid-stride loop covers very large
// batches).  A row needs two passes, maximum then weights; both come from HBM, which is what bounds
// the kernel (2 x 4 bytes per logit at ~4.7 TB/s).  Warps take tiles of 2048 logits (coalesced
// 16-byte loads), tile sums go to shared memory, the tile holding the crossing is scanned in
// element order by one warp.
#include "common.cuh"

namespace reader {

constexpr int kSampleThreads = 256;
constexpr int kSampleTile = 2048;
constexpr int kSampleCand = 2048;
constexpr int kSampleMaxTiles = 1024;   // vocabularies up to 2 Mi entries

// The weight of the definition above, computed without conversion instructions (they run on the slow
// special-function pipe): adding 1.5 * 2^23 rounds x to the nearest integer, ties to even, and leaves
// that integer in the low mantissa bits; trunc(p * 2^(n + 40)) is a shift of p's 24-bit significand.
__device__ __forceinline__ unsigned long long sample_weight(float l, float m, float c) {
    const float x = __fmul_rn(__fsub_rn(l, m), c);
    if (!(x >= -64.0f)) return 0ull;                                  // also NaN
    const float magic = 12582912.0f;                                   // 1.5 * 2^23
    const float shifted = __fadd_rn(x, magic);
    const float n = __fsub_rn(shifted, magic);                         // rint(x), exact for |x| <= 64
    const int ni = __float_as_int(shifted) - 0x4B400000;               // the same integer
    const float f = __fsub_rn(x, n);
    float p = 1.3333558146e-3f;
    p = __fmaf_rn(p, f, 9.6181291076e-3f);
    p = __fmaf_rn(p, f, 5.5504108665e-2f);
    p = __fmaf_rn(p, f, 2.4022650696e-1f);
    p = __fmaf_rn(p, f, 6.9314718056e-1f);
    p = __fmaf_rn(p, f, 1.0f);                                         // in [0.70, 1.42): exponent -1 or 0
    const unsigned bits = __float_as_uint(p);
    const unsigned long long sig = (bits & 0x7FFFFFu) | 0x800000u;     // p = sig * 2^(e - 23)
    const int sh = (int)(bits >> 23) - 127 + ni + 17;                  // p * 2^(n + 40) = sig * 2^sh, sh in [-48, 17]
    return sh >= 0 ? sig << sh : sig >> min(-sh, 63);
}

// Order-preserving key of a logit: a < b  <=>  key(a) < key(b); NaN shares the key of -inf.
__device__ __forceinline__ unsigned sample_key(float l) {
    const unsigned u = __float_as_uint(l == l ? l : -INFINITY);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float sample_unkey(unsigned k) {
    return __uint_as_float((k & 0x80000000u) ? (k & 0x7FFFFFFFu) : ~k);
}

__device__ __forceinline__ unsigned long long warp_sum(unsigned long long v) {
    for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xffffffffu, v, d);
    return v;
}

struct SampleShared {
    float wmax[kSampleThreads / 32];
    float tmax[kSampleThreads];                       // per-thread maxima of the max pass: disjoint subsets of the row
    float u;
    unsigned long long tile_sum[kSampleMaxTiles];
    unsigned long long hist[2048];                    // counts or weight sums per radix digit
    unsigned cand[kSampleCand];                       // keys above the bound
    unsigned n_cand, sel_prefix, bound_key;
    unsigned long long sel_left, total, acc;
};

__global__ void __launch_bounds__(kSampleThreads, 4) sample_kernel(const float *__restrict__ logits, int64_t vocab,
                                                                const int32_t *__restrict__ parent,
                                                                const float *__restrict__ uniforms, int T, float c,
                                                                int64_t rows, int64_t top_k, unsigned top_p_q24,
                                                                int32_t *__restrict__ target) {
    pdl_wait();
    pdl_launch_dependents();
    __shared__ SampleShared sh;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const bool vec = (vocab & 3) == 0;   // rows are then 16-byte aligned (the base pointer is)
    const int n_tiles = (int)((vocab + kSampleTile - 1) / kSampleTile);

    for (int64_t row = blockIdx.x; row < rows; row += gridDim.x) {
        __syncthreads();   // the shared scratch of the previous row is free
        const float *src = logits + row * vocab;

        // ---- block-wide building blocks (every thread calls them; they synchronise inside) ----------
        auto for_each_logit = [&](auto &&f) {   // one streaming pass over the row, four loads in flight
            if (vec) {
                const float4 *v4 = reinterpret_cast<const float4 *>(src);
                const int64_t n4 = vocab / 4;
                int64_t i = tid;
                for (; i + 3 * kSampleThreads < n4; i += 4 * kSampleThreads) {
                    float4 a[4];
#pragma unroll
                    for (int q = 0; q < 4; ++q) a[q] = v4[i + q * kSampleThreads];
#pragma unroll
                    for (int q = 0; q < 4; ++q) { f(a[q].x); f(a[q].y); f(a[q].z); f(a[q].w); }
                }
                for (; i < n4; i += kSampleThreads) {
                    const float4 a = v4[i];
                    f(a.x); f(a.y); f(a.z); f(a.w);
                }
            } else {
                for (int64_t i = tid; i < vocab; i += kSampleThreads) f(src[i]);
            }
        };
        // The k-th largest logit is at least the k-th largest of the per-thread maxima (k distinct
        // logits are that large), so a select for k <= 256 needs only the logits above that bound.
        auto bound_from_maxima = [&](int64_t k) -> unsigned {
            if (tid == 0) sh.bound_key = 0;
            __syncthreads();
            if (k <= kSampleThreads) {
                const float mine = sh.tmax[tid];
                int rank = 0;
                for (int j = 0; j < kSampleThreads; ++j) rank += sh.tmax[j] > mine || (sh.tmax[j] == mine && j < tid);
                if (rank == (int)k - 1) sh.bound_key = sample_key(mine);
            }
            __syncthreads();
            return sh.bound_key;
        };
        // One pass collects the keys >= bound into shared memory; false if they do not fit.
        auto collect = [&](unsigned bound) -> bool {
            if (tid == 0) sh.n_cand = 0;
            __syncthreads();
            for_each_logit([&](float l) {
                const unsigned key = sample_key(l);
                if (key >= bound) {
                    const unsigned at = atomicAdd(&sh.n_cand, 1u);
                    if (at < kSampleCand) sh.cand[at] = key;
                }
            });
            __syncthreads();
            return sh.n_cand <= kSampleCand;
        };
        // Radix select over an order-preserving key, three digits from the top (11 + 11 + 10 bits):
        // the largest key t such that the keys >= t (among those >= floor_key, taken from the candidate
        // list or from the row) count, or weigh, at least `left`.
        auto radix_select = [&](unsigned long long left, bool weighted, bool from_list, unsigned floor_key, float m) -> unsigned {
            if (tid == 0) { sh.sel_prefix = 0; sh.sel_left = left; }
            const int shifts[3] = {21, 10, 0}, widths[3] = {11, 11, 10};
            for (int pass = 0; pass < 3; ++pass) {
                const int shift = shifts[pass], width = widths[pass], nbins = 1 << width;
                for (int i = tid; i < nbins; i += kSampleThreads) sh.hist[i] = 0;
                __syncthreads();
                const unsigned prefix = sh.sel_prefix;          // the digits above this one, already fixed
                auto add = [&](unsigned key) {
                    if (key >= floor_key && (pass == 0 || (key >> (shift + width)) == prefix)) {
                        // a 64-bit sum kept by two 32-bit additions (low word first, its carry into the high
                        // word): exact, and native 32-bit shared-memory atomics instead of a 64-bit one
                        unsigned *bin = reinterpret_cast<unsigned *>(&sh.hist[(key >> shift) & (nbins - 1)]);
                        if (!weighted) {
                            atomicAdd(bin, 1u);                         // at most 2^21 keys: no carry
                        } else {
                            const unsigned long long wgt = sample_weight(sample_unkey(key), m, c);
                            const unsigned lo = (unsigned)wgt, hi = (unsigned)(wgt >> 32);
                            unsigned carry = 0;
                            if (lo) carry = atomicAdd(bin, lo) > ~lo ? 1u : 0u;   // old + lo wrapped
                            if (hi | carry) atomicAdd(bin + 1, hi + carry);
                        }
                    }
                };
                if (from_list) {
                    for (unsigned i = tid; i < sh.n_cand; i += kSampleThreads) add(sh.cand[i]);
                } else {
                    for_each_logit([&](float l) { add(sample_key(l)); });
                }
                __syncthreads();
                if (warp == 0) {   // from the top bin down: the bin in which the running sum reaches what is left
                    const unsigned long long want = sh.sel_left;
                    unsigned long long above = 0;
                    int found = 0;
                    for (int b0 = nbins - 32; b0 >= 0; b0 -= 32) {
                        const unsigned long long cnt = sh.hist[b0 + 31 - lane];   // lane 0 holds the chunk's highest bin
                        unsigned long long incl = cnt;
                        for (int d = 1; d < 32; d <<= 1) {
                            const unsigned long long up = __shfl_up_sync(0xffffffffu, incl, d);
                            if (lane >= d) incl += up;
                        }
                        const unsigned hit = __ballot_sync(0xffffffffu, above + incl >= want);
                        if (hit) {
                            const int first = __ffs(hit) - 1;
                            found = b0 + 31 - first;
                            above += __shfl_sync(0xffffffffu, incl, first) - __shfl_sync(0xffffffffu, cnt, first);
                            break;
                        }
                        above += __shfl_sync(0xffffffffu, incl, 31);
                    }
                    if (lane == 0) {
                        sh.sel_prefix = (prefix << width) | (unsigned)found;
                        sh.sel_left = want - above;
                    }
                }
                __syncthreads();
            }
            return sh.sel_prefix;
        };
        // Integer weights of the logits >= tau, summed per tile of kSampleTile logits (a warp per tile),
        // and their total.
        auto tile_sums = [&](float tau, float m) {
            auto wt = [&](float l) { return l >= tau ? sample_weight(l, m, c) : 0ull; };   // NaN fails the comparison
            for (int t = warp; t < n_tiles; t += kSampleThreads / 32) {
                const int64_t base = (int64_t)t * kSampleTile;
                unsigned long long s = 0;
                if (vec) {
#pragma unroll
                    for (int k0 = 0; k0 < kSampleTile; k0 += 8 * 128) {   // eight loads in flight per lane
                        float4 a[8];
#pragma unroll
                        for (int q = 0; q < 8; ++q) {
                            const int k = k0 + q * 128 + lane * 4;
                            a[q] = base + k < vocab ? *reinterpret_cast<const float4 *>(src + base + k)
                                                    : make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);   // weight 0
                        }
#pragma unroll
                        for (int q = 0; q < 8; ++q) s += wt(a[q].x) + wt(a[q].y) + wt(a[q].z) + wt(a[q].w);
                    }
                } else {
                    for (int k = lane; k < kSampleTile; k += 32)
                        if (base + k < vocab) s += wt(src[base + k]);
                }
                s = warp_sum(s);
                if (lane == 0) sh.tile_sum[t] = s;
            }
            __syncthreads();
            if (warp == 0) {
                unsigned long long total = 0;
                for (int t = lane; t < n_tiles; t += 32) total += sh.tile_sum[t];
                total = warp_sum(total);
                if (lane == 0) sh.total = total;
            }
            __syncthreads();
        };

        // ---- the row ---------------------------------------------------------------------------------
        if (tid == 0) {   // level of this node: its uniform is shared by all nodes of the level
            const int b = (int)(row / T), j = (int)(row % T);
            int lv = 0;
            for (int i = j, steps = 0; i >= 0 && i < T && steps < T; ++steps) {
                ++lv;
                const int up = parent[(size_t)b * T + i];
                i = up < i ? up : -1;   // a malformed parent array cannot send the walk astray
            }
            float u = uniforms[(size_t)b * T + lv - 1];
            if (!(u >= 0.f)) u = 0.f;
            if (u > 0.99999994f) u = 0.99999994f;
            sh.u = u;
        }
        float m = -INFINITY;                                   // row maximum (a NaN never wins)
        for_each_logit([&](float a) { if (a > m) m = a; });
        sh.tmax[tid] = m;
        for (int d = 16; d > 0; d >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, d));
        if (lane == 0) sh.wmax[warp] = m;
        __syncthreads();
        m = sh.wmax[0];
        for (int k = 1; k < kSampleThreads / 32; ++k) m = fmaxf(m, sh.wmax[k]);
        if (m == -INFINITY) {   // nothing has weight (the same m in every thread)
            if (tid == 0) target[row] = 0;
            continue;
        }

        // top-k: tau = the top_k-th largest logit
        float tau = -INFINITY;
        unsigned tau_key = 0, bound = 0;
        bool listed = false;                                   // cand[] holds every key >= bound
        if (top_k > 0 && top_k < vocab) {
            bound = bound_from_maxima(top_k);
            if (bound) listed = collect(bound);
            tau_key = radix_select((unsigned long long)top_k, false, listed, bound, m);
            tau = sample_unkey(tau_key);
        }
        tile_sums(tau, m);

        // top-p: the smallest set of highest logits that weighs at least the requested share
        if (top_p_q24 < (1u << 24) && sh.total > 0) {
            unsigned long long need = (__umul64hi(sh.total, (unsigned long long)top_p_q24) << 40) | ((sh.total * top_p_q24) >> 24);
            if (need == 0) need = 1;
            bool use_list = listed;                            // a list made for top-k holds every kept logit
            if (!listed) {
                // usually the nucleus lies within the logits above the 256th largest per-thread maximum:
                // collect those and check that they weigh enough; otherwise select on the whole row
                bound = bound_from_maxima(kSampleThreads);
                if (bound && collect(bound)) {
                    if (tid == 0) sh.acc = 0;
                    __syncthreads();
                    unsigned long long mine = 0;
                    for (unsigned i = tid; i < sh.n_cand; i += kSampleThreads)
                        if (sh.cand[i] >= tau_key) mine += sample_weight(sample_unkey(sh.cand[i]), m, c);
                    mine = warp_sum(mine);
                    if (lane == 0) atomicAdd(&sh.acc, mine);
                    __syncthreads();
                    use_list = sh.acc >= need;
                }
            }
            const unsigned taup_key = radix_select(need, true, use_list, tau_key, m);
            if (taup_key > tau_key) {
                tau = sample_unkey(taup_key);
                tile_sums(tau, m);
            }
        }

        // ---- threshold, crossing tile, crossing element (warp 0)
        if (warp != 0) continue;
        const unsigned long long total = sh.total;
        if (total == 0) {
            if (lane == 0) target[row] = 0;
            continue;
        }
        auto wt = [&](float l) { return l >= tau ? sample_weight(l, m, c) : 0ull; };
        const unsigned long long U = __float2ull_rz(__fmul_rn(sh.u, 16777216.0f));
        const unsigned long long thr = (__umul64hi(total, U) << 40) | ((total * U) >> 24);
        // tiles in order: the first whose inclusive prefix exceeds thr
        unsigned long long before = 0;
        int tile = n_tiles - 1;
        for (int t0 = 0; t0 < n_tiles; t0 += 32) {
            const int t = t0 + lane;
            const unsigned long long own = t < n_tiles ? sh.tile_sum[t] : 0ull;
            unsigned long long incl = own;
            for (int d = 1; d < 32; d <<= 1) {
                const unsigned long long up = __shfl_up_sync(0xffffffffu, incl, d);
                if (lane >= d) incl += up;
            }
            const unsigned hit = __ballot_sync(0xffffffffu, t < n_tiles && before + incl > thr);
            if (hit) {
                const int first = __ffs(hit) - 1;
                tile = t0 + first;
                before += __shfl_sync(0xffffffffu, incl, first) - __shfl_sync(0xffffffffu, own, first);
                break;
            }
            before += __shfl_sync(0xffffffffu, incl, 31);
        }
        // inside the tile: lane owns 64 consecutive logits
        const int64_t base = (int64_t)tile * kSampleTile + lane * 64;
        unsigned long long mine = 0;
        for (int k = 0; k < 64; ++k)
            if (base + k < vocab) mine += wt(src[base + k]);
        unsigned long long incl = mine;
        for (int d = 1; d < 32; d <<= 1) {
            const unsigned long long up = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= d) incl += up;
        }
        const unsigned hit = __ballot_sync(0xffffffffu, before + incl > thr);
        const int owner = hit ? __ffs(hit) - 1 : 31;
        if (lane == owner) {
            unsigned long long run = before + incl - mine;
            int64_t v = min(base + 63, vocab - 1);
            for (int k = 0; k < 64; ++k) {
                if (base + k >= vocab) break;
                run += wt(src[base + k]);
                if (run > thr) { v = base + k; break; }
            }
            target[row] = (int32_t)v;
        }
    }
}

void launch_sample(const float *logits, int64_t rows, int64_t vocab, const int32_t *parent, const float *uniforms,
                   int T, float c, int64_t top_k, float top_p, int32_t *target, int n_sm, cudaStream_t st) {
    if (rows <= 0) return;
    unsigned q24 = 1u << 24;                                   // off
    if (top_p < 1.0f) {
        if (!(top_p >= 5.9604645e-8f)) top_p = 5.9604645e-8f;  // 2^-24; also NaN
        q24 = (unsigned)(top_p * 16777216.0f);
    }
    const int64_t ctas = rows < 8 * (int64_t)n_sm ? rows : 8 * (int64_t)n_sm;
    launch_pdl(sample_kernel, dim3((unsigned)ctas), dim3(kSampleThreads), 0, st, logits, vocab, parent, uniforms, T, c,
               rows, top_k, q24, target);
}

int sample_max_vocab() { return kSampleTile * kSampleMaxTiles; }

}  // namespace reader
