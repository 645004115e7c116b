// a4: paged causal GQA attention for the rows of one call (Sec. 5.4: attention per sequence
// over its valid KV pages only; Algorithm 2: row j conditions on x, S_{1:j}, i.e. on every
// cached position < p0 plus the in-block rows 0..j).
#pragma once

#include "kernels.cuh"

namespace hispec {

struct AttnArgs {
    const float *q;                // [T][hq*hd] rotated queries
    const __nv_bfloat16 *k_pages;  // [pool_layers][n_pages][hkv][page][hd]
    const __nv_bfloat16 *v_pages;
    const int32_t *block_table;    // [batch][max_pages]
    long long n_pages;
    int pool_layer, hq, hkv, hd;
    float scale;
    __nv_bfloat16 *out;            // [2][T_alloc][hq*hd] hi / lo planes
    int T_alloc, plain;
};

// Straightforward kernel: one warp per (row, query head); lane owns hd/32 consecutive dims;
// keys visited in position order with an online softmax.  Kept as the on-device reference of
// the tiled kernel below.
template <int HD>
__global__ void attention_rowwarp_kernel(StageArgs a, RowMeta rm, AttnArgs p, uint32_t *status) {
    pdl_launch_dependents();
    pdl_wait();
    constexpr int E = HD / 32;
    int gw = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    int t = gw / p.hq, h = gw % p.hq;
    if (t >= a.batch * a.R_pad) return;
    int b = t / a.R_pad, j = t % a.R_pad;
    int nq = p.hq * HD;
    __nv_bfloat16 *ohi = p.out + (size_t)t * nq + h * HD + lane * E;
    __nv_bfloat16 *olo = p.out + ((size_t)p.T_alloc + t) * nq + h * HD + lane * E;
    if (j >= rm.n_rows[b]) {
#pragma unroll
        for (int e = 0; e < E; ++e) { ohi[e] = __float2bfloat16_rn(0.f); olo[e] = __float2bfloat16_rn(0.f); }
        return;
    }
    int kvh = h / (p.hq / p.hkv);
    int n_keys = rm.p0[b] + j + 1;
    float qv[E], acc[E];
#pragma unroll
    for (int e = 0; e < E; ++e) { qv[e] = p.q[(size_t)t * nq + h * HD + lane * E + e] * p.scale; acc[e] = 0.f; }
    float m = -INFINITY, l = 0.f;
    for (int pg = 0; pg * a.page_size < n_keys; ++pg) {
        long long page = p.block_table[(size_t)b * a.max_pages + pg];
        if (page < 0 || page >= p.n_pages) {
            if (lane == 0) atomicOr(status, HISPEC_ST_BOUNDS);
            continue;
        }
        size_t base = ((((size_t)p.pool_layer * p.n_pages + page) * p.hkv + kvh) * a.page_size) * HD;
        int n_in = min(a.page_size, n_keys - pg * a.page_size);
        for (int s = 0; s < n_in; ++s) {
            const __nv_bfloat16 *kp = p.k_pages + base + (size_t)s * HD + lane * E;
            const __nv_bfloat16 *vp = p.v_pages + base + (size_t)s * HD + lane * E;
            float d = 0.f;
#pragma unroll
            for (int e = 0; e < E; ++e) d += qv[e] * __bfloat162float(kp[e]);
            d = warp_sum(d);
            float mn = fmaxf(m, d);
            float corr = expf(m - mn), w = expf(d - mn);
            l = l * corr + w;
#pragma unroll
            for (int e = 0; e < E; ++e) acc[e] = acc[e] * corr + w * __bfloat162float(vp[e]);
            m = mn;
        }
    }
    float inv = 1.0f / l;
#pragma unroll
    for (int e = 0; e < E; ++e) split_hi_lo(acc[e] * inv, ohi[e], olo[e], p.plain);
}

}  // namespace hispec
