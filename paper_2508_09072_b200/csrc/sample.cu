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
// One CTA per row: warps take tiles of 2048 logits (coalesced 16-byte loads), tile sums go to
// shared memory, the tile holding the crossing is scanned in element order by one warp.
#include "common.cuh"

namespace reader {

constexpr int kSampleThreads = 512;
constexpr int kSampleTile = 2048;
constexpr int kSampleMaxTiles = 1024;   // vocabularies up to 2 Mi entries

__device__ __forceinline__ unsigned long long sample_weight(float l, float m, float c) {
    const float x = __fmul_rn(__fsub_rn(l, m), c);
    if (!(x >= -64.0f)) return 0ull;
    const float n = rintf(x);
    const float f = __fsub_rn(x, n);
    float p = 1.3333558146e-3f;
    p = __fmaf_rn(p, f, 9.6181291076e-3f);
    p = __fmaf_rn(p, f, 5.5504108665e-2f);
    p = __fmaf_rn(p, f, 2.4022650696e-1f);
    p = __fmaf_rn(p, f, 6.9314718056e-1f);
    p = __fmaf_rn(p, f, 1.0f);
    const float scale = __int_as_float(((int)n + 40 + 127) << 23);   // 2^(n + 40), exponent in [-24, 40]
    return __float2ull_rz(__fmul_rn(p, scale));                      // exact product, then truncation
}

__device__ __forceinline__ unsigned long long warp_sum(unsigned long long v) {
    for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xffffffffu, v, d);
    return v;
}

__global__ void __launch_bounds__(kSampleThreads) sample_kernel(const float *__restrict__ logits, int64_t vocab,
                                                                const int32_t *__restrict__ parent,
                                                                const float *__restrict__ uniforms, int T, float c,
                                                                int32_t *__restrict__ target) {
    pdl_wait();
    pdl_launch_dependents();
    __shared__ float wmax[kSampleThreads / 32];
    __shared__ unsigned long long tile_sum[kSampleMaxTiles];
    __shared__ float u_s;
    const int64_t row = blockIdx.x;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const float *src = logits + row * vocab;
    const bool vec = (vocab & 3) == 0;   // rows are then 16-byte aligned (the base pointer is)

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
        for (int64_t i = tid; i < vocab / 4; i += kSampleThreads) {
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
    for (int d = 16; d > 0; d >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, d));
    if (lane == 0) wmax[warp] = m;
    __syncthreads();
    m = wmax[0];
    for (int k = 1; k < kSampleThreads / 32; ++k) m = fmaxf(m, wmax[k]);
    if (m == -INFINITY) {   // nothing has weight
        if (tid == 0) target[row] = 0;
        return;
    }

    // ---- integer weights, summed per tile of kSampleTile logits (a warp per tile)
    const int n_tiles = (int)((vocab + kSampleTile - 1) / kSampleTile);
    for (int t = warp; t < n_tiles; t += kSampleThreads / 32) {
        const int64_t base = (int64_t)t * kSampleTile;
        unsigned long long s = 0;
        if (vec) {
            for (int k = lane * 4; k < kSampleTile; k += 128) {
                if (base + k < vocab) {
                    const float4 a = *reinterpret_cast<const float4 *>(src + base + k);
                    s += sample_weight(a.x, m, c) + sample_weight(a.y, m, c) + sample_weight(a.z, m, c) + sample_weight(a.w, m, c);
                }
            }
        } else {
            for (int k = lane; k < kSampleTile; k += 32)
                if (base + k < vocab) s += sample_weight(src[base + k], m, c);
        }
        s = warp_sum(s);
        if (lane == 0) tile_sum[t] = s;
    }
    __syncthreads();

    // ---- threshold, crossing tile, crossing element (warp 0)
    if (warp != 0) return;
    unsigned long long total = 0;
    for (int t = lane; t < n_tiles; t += 32) total += tile_sum[t];
    total = warp_sum(total);
    if (total == 0) {
        if (lane == 0) target[row] = 0;
        return;
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
        if (base + k < vocab) mine += sample_weight(src[base + k], m, c);
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
            run += sample_weight(src[base + k], m, c);
            if (run > thr) { v = base + k; break; }
        }
        target[row] = (int32_t)v;
    }
}

void launch_sample(const float *logits, int64_t rows, int64_t vocab, const int32_t *parent, const float *uniforms,
                   int T, float c, int32_t *target, cudaStream_t st) {
    if (rows <= 0) return;
    launch_pdl(sample_kernel, dim3((unsigned)rows), dim3(kSampleThreads), 0, st, logits, vocab, parent, uniforms, T, c, target);
}

int sample_max_vocab() { return kSampleTile * kSampleMaxTiles; }

}  // namespace reader
