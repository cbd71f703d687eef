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

__global__ void __launch_bounds__(kSampleThreads, 4) sample_kernel(const float *__restrict__ logits, int64_t vocab,
                                                                const int32_t *__restrict__ parent,
                                                                const float *__restrict__ uniforms, int T, float c,
                                                                int64_t rows, int64_t top_k,
                                                                int32_t *__restrict__ target) {
    pdl_wait();
    pdl_launch_dependents();
    __shared__ float wmax[kSampleThreads / 32];
    __shared__ unsigned long long tile_sum[kSampleMaxTiles];
    __shared__ float u_s;
    __shared__ unsigned hist[2048];
    __shared__ unsigned sel_prefix, sel_left, bound_key;
    __shared__ unsigned cand[kSampleCand], n_cand;   // keys above the bound
    __shared__ float tmax[kSampleThreads];   // per-thread maxima of the max pass: disjoint subsets of the row
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const bool vec = (vocab & 3) == 0;   // rows are then 16-byte aligned (the base pointer is)
  for (int64_t row = blockIdx.x; row < rows; row += gridDim.x) {
    __syncthreads();   // the shared scratch of the previous row is free
    const float *src = logits + row * vocab;

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
        u_s = u;
    }

    // ---- row maximum
    float m = -INFINITY;
    if (vec) {
        const float4 *v4 = reinterpret_cast<const float4 *>(src);
        const int64_t n4 = vocab / 4;
        int64_t i = tid;
        for (; i + 3 * kSampleThreads < n4; i += 4 * kSampleThreads) {   // four loads in flight per thread
            float4 a[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) a[q] = v4[i + q * kSampleThreads];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                if (a[q].x > m) m = a[q].x;
                if (a[q].y > m) m = a[q].y;
                if (a[q].z > m) m = a[q].z;
                if (a[q].w > m) m = a[q].w;
            }
        }
        for (; i < n4; i += kSampleThreads) {
            const float4 a = v4[i];
            if (a.x > m) m = a.x;
            if (a.y > m) m = a.y;
            if (a.z > m) m = a.z;
            if (a.w > m) m = a.w;
        }
    } else {
        for (int64_t i = tid; i < vocab; i += kSampleThreads) {
            const float a = src[i];
            if (a > m) m = a;
        }
    }
    tmax[tid] = m;
    for (int d = 16; d > 0; d >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, d));
    if (lane == 0) wmax[warp] = m;
    __syncthreads();
    m = wmax[0];
    for (int k = 1; k < kSampleThreads / 32; ++k) m = fmaxf(m, wmax[k]);
    if (m == -INFINITY) {   // nothing has weight (the same m in every thread)
        if (tid == 0) target[row] = 0;
        continue;
    }

    // ---- top-k threshold: radix select of the top_k-th largest key
    float tau = -INFINITY;
    if (top_k > 0 && top_k < vocab) {
        if (tid == 0) { sel_prefix = 0; sel_left = (unsigned)top_k; bound_key = 0; }
        __syncthreads();
        // The k-th largest logit is at least the k-th largest of the per-thread maxima (k distinct
        // logits are at least that large), so nothing below it needs counting: for the usual small k
        // only a few hundred of the row's logits take part in the select.
        if (top_k <= kSampleThreads) {
            const float mine = tmax[tid];
            int rank = 0;
            for (int j = 0; j < kSampleThreads; ++j) rank += tmax[j] > mine || (tmax[j] == mine && j < tid);
            if (rank == (int)top_k - 1) bound_key = sample_key(mine);
        }
        __syncthreads();
        const unsigned bound = bound_key;
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
        // With a bound, one pass collects the keys above it (a few hundred) and the select runs on
        // that list in shared memory; without one (or if the list overflows) it runs on the row.
        bool listed = false;
        if (bound != 0) {
            if (tid == 0) n_cand = 0;
            __syncthreads();
            for_each_logit([&](float l) {
                const unsigned key = sample_key(l);
                if (key >= bound) {
                    const unsigned at = atomicAdd(&n_cand, 1u);
                    if (at < kSampleCand) cand[at] = key;
                }
            });
            __syncthreads();
            listed = n_cand <= kSampleCand;
        }
        const int shifts[3] = {21, 10, 0}, widths[3] = {11, 11, 10};
        for (int pass = 0; pass < 3; ++pass) {
            const int shift = shifts[pass], nbins = 1 << widths[pass];
            for (int i = tid; i < nbins; i += kSampleThreads) hist[i] = 0;
            __syncthreads();
            const unsigned prefix = sel_prefix;                 // the bits above this digit, already fixed
            auto count = [&](unsigned key) {
                if (key >= bound && (pass == 0 || (key >> (shift + widths[pass])) == prefix))
                    atomicAdd(&hist[(key >> shift) & (nbins - 1)], 1u);
            };
            if (listed) {
                for (unsigned i = tid; i < n_cand; i += kSampleThreads) count(cand[i]);
            } else {
                for_each_logit([&](float l) { count(sample_key(l)); });
            }
            __syncthreads();
            if (warp == 0) {   // from the top bin down: the bin in which the count reaches what is left
                unsigned left = sel_left, above = 0;
                int found = 0;
                for (int b0 = nbins - 32; b0 >= 0; b0 -= 32) {
                    const unsigned c = hist[b0 + 31 - lane];    // lane 0 holds the highest bin of the chunk
                    unsigned incl = c;
                    for (int d = 1; d < 32; d <<= 1) {
                        const unsigned up = __shfl_up_sync(0xffffffffu, incl, d);
                        if (lane >= d) incl += up;
                    }
                    const unsigned hit = __ballot_sync(0xffffffffu, above + incl >= left);
                    if (hit) {
                        const int first = __ffs(hit) - 1;
                        found = b0 + 31 - first;
                        above += __shfl_sync(0xffffffffu, incl, first) - __shfl_sync(0xffffffffu, c, first);
                        break;
                    }
                    above += __shfl_sync(0xffffffffu, incl, 31);
                }
                if (lane == 0) {
                    sel_prefix = (prefix << widths[pass]) | (unsigned)found;
                    sel_left = left - above;
                }
            }
            __syncthreads();
        }
        tau = sample_unkey(sel_prefix);
    }
    // a logit keeps its weight iff it is at least tau (NaN fails the comparison)
#define SAMPLE_W(l) ((l) >= tau ? sample_weight((l), m, c) : 0ull)

    // ---- integer weights, summed per tile of kSampleTile logits (a warp per tile)
    const int n_tiles = (int)((vocab + kSampleTile - 1) / kSampleTile);
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
                    a[q] = base + k < vocab ? __ldcs(reinterpret_cast<const float4 *>(src + base + k))   // last use of the row
                                            : make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);  // weight 0
                }
#pragma unroll
                for (int q = 0; q < 8; ++q)
                    s += SAMPLE_W(a[q].x) + SAMPLE_W(a[q].y) + SAMPLE_W(a[q].z) + SAMPLE_W(a[q].w);
            }
        } else {
            for (int k = lane; k < kSampleTile; k += 32)
                if (base + k < vocab) s += SAMPLE_W(src[base + k]);
        }
        s = warp_sum(s);
        if (lane == 0) tile_sum[t] = s;
    }
    __syncthreads();

    // ---- threshold, crossing tile, crossing element (warp 0)
    if (warp != 0) continue;
    unsigned long long total = 0;
    for (int t = lane; t < n_tiles; t += 32) total += tile_sum[t];
    total = warp_sum(total);
    if (total == 0) {
        if (lane == 0) target[row] = 0;
        continue;
    }
    const unsigned long long U = __float2ull_rz(__fmul_rn(u_s, 16777216.0f));
    const unsigned long long thr = (__umul64hi(total, U) << 40) | ((total * U) >> 24);
    // tiles in order: the first whose inclusive prefix exceeds thr
    unsigned long long before = 0;
    int tile = n_tiles - 1;
    for (int t0 = 0; t0 < n_tiles; t0 += 32) {
        const int t = t0 + lane;
        unsigned long long incl = t < n_tiles ? tile_sum[t] : 0;
        for (int d = 1; d < 32; d <<= 1) {
            const unsigned long long up = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= d) incl += up;
        }
        const unsigned hit = __ballot_sync(0xffffffffu, t < n_tiles && before + incl > thr);
        if (hit) {
            const int first = __ffs(hit) - 1;
            const unsigned long long excl = __shfl_sync(0xffffffffu, incl, first) - __shfl_sync(0xffffffffu, t < n_tiles ? tile_sum[t] : 0ull, first);
            tile = t0 + first;
            before += excl;
            break;
        }
        before += __shfl_sync(0xffffffffu, incl, 31);
    }
    // inside the tile: lane owns 64 consecutive logits
    const int64_t base = (int64_t)tile * kSampleTile + lane * 64;
    unsigned long long mine = 0;
    for (int k = 0; k < 64; ++k)
        if (base + k < vocab) mine += SAMPLE_W(src[base + k]);
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
            run += SAMPLE_W(src[base + k]);
            if (run > thr) { v = base + k; break; }
        }
        target[row] = (int32_t)v;
    }
  }
}

void launch_sample(const float *logits, int64_t rows, int64_t vocab, const int32_t *parent, const float *uniforms,
                   int T, float c, int64_t top_k, int32_t *target, int n_sm, cudaStream_t st) {
    if (rows <= 0) return;
    const int64_t ctas = rows < 8 * (int64_t)n_sm ? rows : 8 * (int64_t)n_sm;
    launch_pdl(sample_kernel, dim3((unsigned)ctas), dim3(kSampleThreads), 0, st, logits, vocab, parent, uniforms, T, c, rows, top_k, target);
}

#undef SAMPLE_W
int sample_max_vocab() { return kSampleTile * kSampleMaxTiles; }

}  // namespace reader
