// Split-KV combine: merges the (m, l, O) partials of every unit that was cut across CTA ranges,
//   m* = max_s m_s,  l* = sum_s l_s 2^(m_s - m*),  O = sum_s O_s 2^(m_s - m*) / l*,
// rounds to bf16 and writes lse = ln 2 * (m* + log2 l*).  Units written directly by the attention
// kernel are left alone; rows of sequences with a non-zero status are zeroed, and so is every row when the
// attention kernel raised the error flag (each status word then carries that code).
#include "common.cuh"

namespace reader {

__global__ void __launch_bounds__(128) combine_kernel(const AttnParams p) {
    const int unit_global = blockIdx.x;
    const int ups = p.sched.units_per_seq;
    const int b = unit_global / ups;
    const int unit = unit_global - b * ups;
    const int h = unit / p.sched.n_mtiles;
    const int mt = unit - h * p.sched.n_mtiles;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int row = blockIdx.y * 4 + warp;   // one warp per query row: the merge is latency-bound, so spread it wide
    const int D = p.D;
    const int nt = p.sched.seq_ntiles[b];
    const int rows = min(kTileM, p.T * p.G - mt * kTileM);

    const int err = *p.error_flag;   // a bounded wait gave up somewhere: no row of this call can be trusted
    if (err != 0 && unit == 0 && blockIdx.y == 0 && threadIdx.x == 0) p.status[b] = err;
    if (nt == 0 || err != 0) {
        if (row < rows) {
            const int grow = mt * kTileM + row;
            const int j = grow / p.G, hq = h * p.G + grow % p.G;
            __nv_bfloat16 *dst = p.out + (((size_t)b * p.T + j) * p.Hq + hq) * D;
            if (lane * 4 < D) *reinterpret_cast<uint2 *>(dst + lane * 4) = make_uint2(0, 0);
            if (p.lse && lane == 0) p.lse[((size_t)b * p.T + j) * p.Hq + hq] = 0.f;
        }
        return;
    }
    const int W = p.sched.seq_tile_start[p.B];
    const int u0 = p.sched.seq_tile_start[b] + unit * nt;
    const int c_first = cta_of_tile(u0, p.sched.n_ctas, W);
    const int c_last = cta_of_tile(u0 + nt - 1, p.sched.n_ctas, W);
    if (c_first == c_last || row >= rows) return;

    {
        const int r = row;
        float mstar = -INFINITY;
        for (int c = c_first; c <= c_last; ++c) {
            if (range_begin(c + 1, p.sched.n_ctas, W) == range_begin(c, p.sched.n_ctas, W)) continue;  // empty range: wrote nothing
            const int slot = c == c_first ? 2 * c + 1 : 2 * c;
            mstar = fmaxf(mstar, p.partial_ml[((size_t)slot * kTileM + r) * 2]);
        }
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        float lstar = 0.f;
        for (int c = c_first; c <= c_last; ++c) {
            if (range_begin(c + 1, p.sched.n_ctas, W) == range_begin(c, p.sched.n_ctas, W)) continue;
            const int slot = c == c_first ? 2 * c + 1 : 2 * c;
            const float2 ml = *reinterpret_cast<const float2 *>(p.partial_ml + ((size_t)slot * kTileM + r) * 2);
            const float wgt = ml.x == -INFINITY ? 0.f : exp2f(ml.x - mstar);
            lstar += ml.y * wgt;
            if (lane * 4 < D) {
                const float4 o = *reinterpret_cast<const float4 *>(p.partial_o + ((size_t)slot * kTileM + r) * D + lane * 4);
                acc.x = fmaf(o.x, wgt, acc.x);
                acc.y = fmaf(o.y, wgt, acc.y);
                acc.z = fmaf(o.z, wgt, acc.z);
                acc.w = fmaf(o.w, wgt, acc.w);
            }
        }
        const float inv = 1.f / lstar;
        const int grow = mt * kTileM + r;
        const int j = grow / p.G, hq = h * p.G + grow % p.G;
        __nv_bfloat16 *dst = p.out + (((size_t)b * p.T + j) * p.Hq + hq) * D;
        if (lane * 4 < D) {
            __nv_bfloat162 a = __floats2bfloat162_rn(acc.x * inv, acc.y * inv);
            __nv_bfloat162 c2 = __floats2bfloat162_rn(acc.z * inv, acc.w * inv);
            uint2 v;
            v.x = *reinterpret_cast<uint32_t *>(&a);
            v.y = *reinterpret_cast<uint32_t *>(&c2);
            *reinterpret_cast<uint2 *>(dst + lane * 4) = v;
        }
        if (p.lse && lane == 0)
            p.lse[((size_t)b * p.T + j) * p.Hq + hq] = (mstar + log2f(lstar)) * 0.6931471805599453f;
    }
}

void launch_combine(const AttnParams &p, cudaStream_t st) {
    const int units = p.B * p.sched.units_per_seq;
    if (units > 0) combine_kernel<<<dim3(units, kTileM / 4), 128, 0, st>>>(p);
}

}  // namespace reader
