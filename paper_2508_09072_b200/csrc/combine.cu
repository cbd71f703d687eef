// Split-KV combine: merges the (m, l, O) partials of every unit that was cut across CTA ranges,
//   m* = max_s m_s,  l* = sum_s l_s 2^(m_s - m*),  O = sum_s O_s 2^(m_s - m*) / l*,
// rounds to bf16 and writes lse = ln 2 * (m* + log2 l*).  Units written directly by the attention
// kernel are left alone.
//
// The work is found without searching: the attention CTA that started a cut unit left a descriptor
// (unit, last CTA) in the workspace, so the four blocks (c, 0..3) read descriptor c and merge 32
// of the unit's 128 rows each, two per warp with their loads in flight together.  If the
// attention kernel raised the error flag (a bounded wait gave up), no row of the call can be
// trusted: everything is zeroed and every status word gets the code.
#include "common.cuh"

namespace reader {

constexpr int kCombineWarps = 16;
constexpr int kRowGroups = 4;                           // blocks per attention CTA, 32 rows each
constexpr int kRowsPerWarp = kTileM / (kCombineWarps * kRowGroups);   // 2 rows: one batch
constexpr int kBatch = 2;

__global__ void __launch_bounds__(kCombineWarps * 32, 2) combine_kernel(const AttnParams p) {
    asm volatile("griddepcontrol.wait;" ::: "memory");   // launched ahead of the attention kernel's end
    const int c0 = blockIdx.x;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int D = p.D;
    const int err = *p.error_flag;
    const SplitDesc d = p.split_desc[c0];
    const int W = p.sched.seq_tile_start[p.B];

    if (err != 0) {
        const size_t nthreads = (size_t)gridDim.x * gridDim.y * blockDim.x;
        const size_t me = ((size_t)blockIdx.y * gridDim.x + blockIdx.x) * blockDim.x + threadIdx.x;
        uint4 *o = reinterpret_cast<uint4 *>(p.out);
        for (size_t i = me; i < (size_t)p.B * p.T * p.Hq * D / 8; i += nthreads) o[i] = make_uint4(0, 0, 0, 0);
        if (p.lse)
            for (size_t i = me; i < (size_t)p.B * p.T * p.Hq; i += nthreads) p.lse[i] = 0.f;
        for (size_t i = me; i < (size_t)p.B; i += nthreads) p.status[i] = err;
        return;
    }
    if (p.zero_rejected) {   // block-uniform loop: every block takes some of the sequences
        const int nblocks = gridDim.x * gridDim.y, me = blockIdx.y * gridDim.x + blockIdx.x;
        for (int b = me; b < p.B; b += nblocks) {
            if (p.status[b] == READER_OK) continue;
            uint4 *o = reinterpret_cast<uint4 *>(p.out + (size_t)b * p.T * p.Hq * D);
            for (size_t i = threadIdx.x; i < (size_t)p.T * p.Hq * D / 8; i += blockDim.x) o[i] = make_uint4(0, 0, 0, 0);
            if (p.lse)
                for (int i = threadIdx.x; i < p.T * p.Hq; i += blockDim.x) p.lse[(size_t)b * p.T * p.Hq + i] = 0.f;
        }
    }
    if (d.b < 0) return;
    const int rows = min(kTileM, p.T * p.G - d.mt * kTileM);
    const bool has_cols = lane * 4 < D;
    const int nm = p.sched.n_mtiles;
    const int n_lanes = effective_ctas(p.sched.n_ctas / nm, W);
    const bool all_live = !p.sched.aligned && W >= n_lanes;   // with fewer tiles than CTAs some ranges are empty

    for (int rb = 0; rb < kRowsPerWarp; rb += kBatch) {
        const int r0 = (blockIdx.y * kCombineWarps + warp) * kRowsPerWarp + rb;
        if (r0 >= rows) break;
        float mstar[kBatch], lstar[kBatch];
        float4 acc[kBatch];
#pragma unroll
        for (int q = 0; q < kBatch; ++q) {
            mstar[q] = -INFINITY; lstar[q] = 0.f;
            acc[q] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
        // online merge over the CTAs c0 .. c_last, two slots x kBatch rows per round of loads
        // the unit's partials sit in the CTAs with the same M tile in the lanes c0 / nm .. c_last / nm
        for (int cb = c0; cb <= d.c_last; cb += 2 * nm) {
            float2 ml[2][kBatch];
            float4 o[2][kBatch];
#pragma unroll
            for (int k = 0; k < 2; ++k) {
                const int c = cb + k * nm;
                // a CTA with an empty range wrote nothing
                bool live = c <= d.c_last;
                if (live && !all_live) {
                    const LaneRange r = lane_range(p.sched, p.B, c / nm, n_lanes, W);
                    live = r.w_end > r.w_begin;
                }
                const int slot = c == c0 ? 2 * c + 1 : 2 * c;
#pragma unroll
                for (int q = 0; q < kBatch; ++q) {
                    const int r = min(r0 + q, kTileM - 1);
                    ml[k][q] = make_float2(-INFINITY, 0.f);
                    o[k][q] = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (live) {
                        ml[k][q] = *reinterpret_cast<const float2 *>(p.partial_ml + ((size_t)slot * kTileM + r) * 2);
                        if (has_cols) o[k][q] = *reinterpret_cast<const float4 *>(p.partial_o + ((size_t)slot * kTileM + r) * D + lane * 4);
                    }
                }
            }
#pragma unroll
            for (int q = 0; q < kBatch; ++q) {
                const float mnew = fmaxf(mstar[q], fmaxf(ml[0][q].x, ml[1][q].x));
                if (mnew == -INFINITY) continue;   // nothing seen yet
                const float keep = mstar[q] == -INFINITY ? 0.f : exp2f(mstar[q] - mnew);
                lstar[q] *= keep;
                acc[q].x *= keep; acc[q].y *= keep; acc[q].z *= keep; acc[q].w *= keep;
#pragma unroll
                for (int k = 0; k < 2; ++k) {
                    const float wgt = ml[k][q].x == -INFINITY ? 0.f : exp2f(ml[k][q].x - mnew);
                    lstar[q] = fmaf(ml[k][q].y, wgt, lstar[q]);
                    acc[q].x = fmaf(o[k][q].x, wgt, acc[q].x);
                    acc[q].y = fmaf(o[k][q].y, wgt, acc[q].y);
                    acc[q].z = fmaf(o[k][q].z, wgt, acc[q].z);
                    acc[q].w = fmaf(o[k][q].w, wgt, acc[q].w);
                }
                mstar[q] = mnew;
            }
        }
#pragma unroll
        for (int q = 0; q < kBatch; ++q) {
            const int r = r0 + q;
            if (r >= rows) break;
            const float inv = 1.f / lstar[q];
            const int grow = d.mt * kTileM + r;
            const int j = grow / p.G, hq = d.h * p.G + grow % p.G;
            __nv_bfloat16 *dst = p.out + (((size_t)d.b * p.T + j) * p.Hq + hq) * D;
            if (has_cols) {
                __nv_bfloat162 a = __floats2bfloat162_rn(acc[q].x * inv, acc[q].y * inv);
                __nv_bfloat162 c2 = __floats2bfloat162_rn(acc[q].z * inv, acc[q].w * inv);
                uint2 v;
                v.x = *reinterpret_cast<uint32_t *>(&a);
                v.y = *reinterpret_cast<uint32_t *>(&c2);
                *reinterpret_cast<uint2 *>(dst + lane * 4) = v;
            }
            if (p.lse && lane == 0)
                p.lse[((size_t)d.b * p.T + j) * p.Hq + hq] = (mstar[q] + log2f(lstar[q])) * 0.6931471805599453f;
        }
    }
}

void launch_combine(const AttnParams &p, cudaStream_t st) {
    if (p.B <= 0) return;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(p.sched.n_ctas, kRowGroups);
    cfg.blockDim = dim3(kCombineWarps * 32);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaLaunchKernelEx(&cfg, combine_kernel, p);
}

}  // namespace reader
