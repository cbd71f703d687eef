// Tree-masked verify attention (Sec. 3.2), shape-generic CUDA-core version: any GQA group size,
// head_dim 64 or 128.  One thread owns one query row (node, group member); K/V tiles of 64 keys
// are staged in shared memory and broadcast to all rows; scores, online softmax and the value
// product are fp32.  It walks the same flattened split-KV partition and writes the same partial
// format as the tensor-core kernel, and serves the shapes that kernel is not built for.
#include "common.cuh"

namespace reader {

template <int D>
__global__ void __launch_bounds__(kTileM) attn_generic_kernel(const AttnParams p) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    uint4 *ks = reinterpret_cast<uint4 *>(smem_raw);                    // [64][D] bf16
    uint4 *vs = reinterpret_cast<uint4 *>(smem_raw + kPage * D * 2);    // [64][D] bf16
    constexpr int kChunks = D / 8;                                      // 16-byte chunks per row

    const int cta = blockIdx.x, tid = threadIdx.x;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int W = p.sched.seq_tile_start[p.B];
    const CtaWork cw = cta_work(p.sched, p.B, cta, W);
    const int w_end = cw.w_end;
    int w = cw.w_begin;
    if (tid == 0) p.split_desc[cta].b = -1;

    while (w < w_end) {
        const Segment sg = segment_at(p.sched, p.B, cta, w, w_end);
        if (tid == 0) record_split(p.split_desc, p.sched, p.B, cw.n_lanes, sg, cta, W);
        w += sg.span;
        if (sg.tile_end <= sg.tile_begin) continue;   // the range ended among the unit's overhead entries

        const int grow = sg.mt * kTileM + tid;           // row within the (b, h) problem
        const bool row_ok = grow < p.T * p.G;
        const int j = row_ok ? grow / p.G : 0;
        const int hq = sg.h * p.G + (row_ok ? grow % p.G : 0);
        const int L = committed_len(p, sg.b);

        uint32_t qreg[D / 2];
        {
            const uint4 *src = reinterpret_cast<const uint4 *>(p.q + (((size_t)sg.b * p.T + j) * p.Hq + hq) * D);
#pragma unroll
            for (int c = 0; c < kChunks; ++c) {
                uint4 v = row_ok ? src[c] : make_uint4(0, 0, 0, 0);
                qreg[4 * c + 0] = v.x; qreg[4 * c + 1] = v.y; qreg[4 * c + 2] = v.z; qreg[4 * c + 3] = v.w;
            }
        }
        const uint64_t anc_lo = p.anc[((size_t)sg.b * p.T + j) * 2 + 0];
        const uint64_t anc_hi = p.anc[((size_t)sg.b * p.T + j) * 2 + 1];

        float o[D];
#pragma unroll
        for (int d = 0; d < D; ++d) o[d] = 0.f;
        float m = -INFINITY, l = 0.f;

        for (int t = sg.tile_begin; t < sg.tile_end; ++t) {
            // ---- stage the tile
            uint64_t vis;
            __syncthreads();
            if (t < sg.npages) {
                const int page = p.valid_bits ? 0 : p.page_table[(size_t)sg.b * p.max_pages + t];
                vis = page_visible(p, sg.b, t, L);
                const size_t base = (size_t)page_first_row(p, sg.b, sg.h, t, page) * D;
                const uint4 *ksrc = reinterpret_cast<const uint4 *>(p.k_pool + base);
                const uint4 *vsrc = reinterpret_cast<const uint4 *>(p.v_pool + base);
                for (int c = tid; c < kPage * kChunks; c += kTileM) {
                    const bool in = (vis >> (c / kChunks)) & 1ull;   // rows no query may see are never read
                    ks[c] = in ? ksrc[c] : make_uint4(0, 0, 0, 0);
                    vs[c] = in ? vsrc[c] : make_uint4(0, 0, 0, 0);
                }
            } else {
                const int kt = t - sg.npages;
                for (int c = tid; c < kPage * kChunks; c += kTileM) {
                    const int node = kt * kPage + c / kChunks;
                    const bool in = node < p.T;
                    const size_t at = (((size_t)sg.b * p.T + node) * p.Hkv + sg.h) * D;
                    ks[c] = in ? reinterpret_cast<const uint4 *>(p.k_tree + at)[c % kChunks] : make_uint4(0, 0, 0, 0);
                    vs[c] = in ? reinterpret_cast<const uint4 *>(p.v_tree + at)[c % kChunks] : make_uint4(0, 0, 0, 0);
                }
                vis = kt == 0 ? anc_lo : anc_hi;   // bits of nodes >= T are never set
            }
            __syncthreads();

            // ---- 16 keys at a time: scores, running max, probabilities, value product
            for (int kb = 0; kb < kPage; kb += 16) {
                const uint32_t vis16 = (uint32_t)(vis >> kb) & 0xffffu;
                if (vis16 == 0) continue;                      // per-thread skip, no barrier inside
                float s[16];
                float bmax = -INFINITY;
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    float acc = 0.f;
                    const uint4 *kr = ks + (kb + i) * kChunks;
#pragma unroll
                    for (int c = 0; c < kChunks; ++c) {
                        const uint4 kv = kr[c];
                        acc = fmaf(bf16lo(qreg[4 * c + 0]), bf16lo(kv.x), acc);
                        acc = fmaf(bf16hi(qreg[4 * c + 0]), bf16hi(kv.x), acc);
                        acc = fmaf(bf16lo(qreg[4 * c + 1]), bf16lo(kv.y), acc);
                        acc = fmaf(bf16hi(qreg[4 * c + 1]), bf16hi(kv.y), acc);
                        acc = fmaf(bf16lo(qreg[4 * c + 2]), bf16lo(kv.z), acc);
                        acc = fmaf(bf16hi(qreg[4 * c + 2]), bf16hi(kv.z), acc);
                        acc = fmaf(bf16lo(qreg[4 * c + 3]), bf16lo(kv.w), acc);
                        acc = fmaf(bf16hi(qreg[4 * c + 3]), bf16hi(kv.w), acc);
                    }
                    s[i] = ((vis16 >> i) & 1u) ? acc * p.scale_log2 : -INFINITY;
                    bmax = fmaxf(bmax, s[i]);
                }
                const float m_new = fmaxf(m, bmax);            // finite: some key of the block is visible
                const float alpha = exp2f(m - m_new);          // m = -inf -> 0
                l *= alpha;
#pragma unroll
                for (int d = 0; d < D; ++d) o[d] *= alpha;
                m = m_new;
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const float pr = exp2f(s[i] - m);
                    l += pr;
                    const uint4 *vr = vs + (kb + i) * kChunks;
#pragma unroll
                    for (int c = 0; c < kChunks; ++c) {
                        const uint4 vv = vr[c];
                        o[8 * c + 0] = fmaf(pr, bf16lo(vv.x), o[8 * c + 0]);
                        o[8 * c + 1] = fmaf(pr, bf16hi(vv.x), o[8 * c + 1]);
                        o[8 * c + 2] = fmaf(pr, bf16lo(vv.y), o[8 * c + 2]);
                        o[8 * c + 3] = fmaf(pr, bf16hi(vv.y), o[8 * c + 3]);
                        o[8 * c + 4] = fmaf(pr, bf16lo(vv.z), o[8 * c + 4]);
                        o[8 * c + 5] = fmaf(pr, bf16hi(vv.z), o[8 * c + 5]);
                        o[8 * c + 6] = fmaf(pr, bf16lo(vv.w), o[8 * c + 6]);
                        o[8 * c + 7] = fmaf(pr, bf16hi(vv.w), o[8 * c + 7]);
                    }
                }
            }
        }

        // ---- segment epilogue
        if (sg.full) {
            if (row_ok) {
                const float inv = 1.f / l;   // l > 0: every node sees itself
                uint4 *dst = reinterpret_cast<uint4 *>(p.out + (((size_t)sg.b * p.T + j) * p.Hq + hq) * D);
#pragma unroll
                for (int c = 0; c < kChunks; ++c) {
                    __nv_bfloat162 a = __floats2bfloat162_rn(o[8 * c + 0] * inv, o[8 * c + 1] * inv);
                    __nv_bfloat162 b2 = __floats2bfloat162_rn(o[8 * c + 2] * inv, o[8 * c + 3] * inv);
                    __nv_bfloat162 c2 = __floats2bfloat162_rn(o[8 * c + 4] * inv, o[8 * c + 5] * inv);
                    __nv_bfloat162 d2 = __floats2bfloat162_rn(o[8 * c + 6] * inv, o[8 * c + 7] * inv);
                    uint4 v;
                    v.x = *reinterpret_cast<uint32_t *>(&a);
                    v.y = *reinterpret_cast<uint32_t *>(&b2);
                    v.z = *reinterpret_cast<uint32_t *>(&c2);
                    v.w = *reinterpret_cast<uint32_t *>(&d2);
                    dst[c] = v;
                }
                if (p.lse) p.lse[((size_t)sg.b * p.T + j) * p.Hq + hq] = (m + log2f(l)) * 0.6931471805599453f;
            }
        } else {
            float4 *po = reinterpret_cast<float4 *>(p.partial_o + ((size_t)sg.slot * kTileM + tid) * D);
#pragma unroll
            for (int c = 0; c < D / 4; ++c) po[c] = make_float4(o[4 * c], o[4 * c + 1], o[4 * c + 2], o[4 * c + 3]);
            float2 *pm = reinterpret_cast<float2 *>(p.partial_ml + ((size_t)sg.slot * kTileM + tid) * 2);
            *pm = make_float2(m, l);
        }
    }
}

void launch_attn_generic(const AttnParams &p, cudaStream_t st) {
    const size_t smem = 2 * kPage * p.D * 2;
    if (p.D == 128)
        attn_generic_kernel<128><<<p.sched.n_ctas, kTileM, smem, st>>>(p);
    else
        attn_generic_kernel<64><<<p.sched.n_ctas, kTileM, smem, st>>>(p);
}

}  // namespace reader
