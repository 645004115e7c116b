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

// ---------------------------------------------------------------------------------------------
// Tiled kernel.  One CTA per (key split, KV head x group of <= 64 stacked query rows, sequence).
// The query rows of all q heads that share the KV head are stacked (row r = j * G + g: block row
// j, head g of the group), so a K/V page is fetched once for all of them.  A producer warp walks
// the block table and stages whole pages (16 keys) with TMA into 128-byte-swizzled shared memory;
// each consumer warp owns 16 stacked rows: S = Q K^T with mma.sync (Q as bf16 hi + lo, so scores
// keep fp32-like accuracy), online softmax in registers with quad shuffles, O += P V.  Each split
// writes an unnormalised (O, m, l) record; attention_merge_kernel combines the splits in a fixed
// order.  Needs page_size == 16.
struct AttnTcArgs {
    const float *q;
    const int32_t *block_table;
    long long n_pages;
    int pool_layer, hq, hkv, G, n_splits, n_mg, mt;
    float scale_log2;  // softmax scale * log2(e)
    float *part;       // [T][hq][n_splits][HD + 2]
};

constexpr int kAttnStages = 4;
// stacked query rows (G x R_pad) one CTA takes: up to eight 16-row warp tiles share every K / V page the CTA stages
constexpr int kAttnGroupRows = 128;

__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
    __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t *>(&v);
}
__device__ __forceinline__ void mma_bf16_16816(float *c, const uint32_t *a, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t *r) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t *r) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
// shared-memory helpers (same PTX as the projection kernel's; kept local so that this header stands alone)
__device__ __forceinline__ uint32_t a_smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ uint32_t a_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok;
}
__device__ __forceinline__ bool a_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, uint32_t *status) {
    for (uint32_t it = 0; it < (1u << 24); ++it) {
        if (a_try_wait(bar, parity)) return true;
        if ((it & 1023u) == 1023u && *abort_flag) return false;
    }
    *abort_flag = 1;
    atomicOr(status, HISPEC_ST_TIMEOUT);
    return false;
}

template <int HD>
__global__ void __launch_bounds__((kAttnGroupRows / 16 + 1) * 32)
attention_tc_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV, StageArgs a,
                    RowMeta rm, AttnTcArgs p, uint32_t *status) {
    constexpr int TILE = 16 * HD * 2;           // bytes of one K (or V) page of one KV head
    constexpr int KS = HD / 16;                 // k-steps of Q K^T
    constexpr int NT = HD / 8;                  // n-tiles of P V
    __shared__ __align__(1024) uint8_t sm[kAttnStages * 2 * TILE];
    __shared__ __align__(8) uint64_t bar_full[kAttnStages], bar_empty[kAttnStages];
    __shared__ int s_abort, s_seq;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int split = blockIdx.x, kvh = blockIdx.y / p.n_mg, mg = blockIdx.y % p.n_mg;
    volatile int *abort_flag = &s_abort;
    if (threadIdx.x == 0) {
        s_abort = 0;
        for (int s = 0; s < kAttnStages; ++s) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(a_smem_u32(&bar_full[s])), "r"(1) : "memory");
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(a_smem_u32(&bar_empty[s])), "r"(p.mt) : "memory");
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    pdl_launch_dependents();
    pdl_wait();

    // blockIdx.z counts the sequences from the longest to the shortest: blocks are dispatched in index order, so the
    // long sequences of a ragged batch start first and the short ones fill the tail
    for (int i = threadIdx.x; i < a.batch; i += blockDim.x) {
        const int li = rm.p0[i] + rm.n_rows[i];
        int rank = 0;
        for (int j = 0; j < a.batch; ++j) {
            const int lj = rm.p0[j] + rm.n_rows[j];
            rank += (lj > li || (lj == li && j < i)) ? 1 : 0;
        }
        if (rank == (int)blockIdx.z) s_seq = i;
    }
    __syncthreads();
    const int b = s_seq;
    const int nr = rm.n_rows[b], p0 = rm.p0[b];
    const int n_keys = p0 + nr;
    const int total_pages = (n_keys + 15) >> 4;
    int chunk = (total_pages + p.n_splits - 1) / p.n_splits;
    if (chunk < 1) chunk = 1;
    const int pg0 = split * chunk;
    const int pg1 = min(pg0 + chunk, total_pages);
    const int n_pg = (nr > 0 && pg1 > pg0) ? pg1 - pg0 : 0;
    const int QR = p.G * a.R_pad;
    const uint32_t sm0 = a_smem_u32(sm);

    if (warp == p.mt) {
        // ---- producer: block-table walk + TMA page loads
        for (int i0 = 0; i0 < n_pg; i0 += 32) {
            int my = i0 + lane;
            long long pgid = 0;
            if (my < n_pg) pgid = p.block_table[(size_t)b * a.max_pages + pg0 + my];
            bool bad = my < n_pg && (pgid < 0 || pgid >= p.n_pages);
            if (bad) { atomicOr(status, HISPEC_ST_BOUNDS); pgid = 0; }
            int cnt = min(32, n_pg - i0);
            for (int u = 0; u < cnt; ++u) {
                long long page = __shfl_sync(0xffffffffu, pgid, u);
                int i = i0 + u;
                int s = i % kAttnStages;
                uint32_t ph = (uint32_t)(i / kAttnStages) & 1u;
                bool ok = true;
                if (lane == 0) {
                    ok = a_wait(a_smem_u32(&bar_empty[s]), ph ^ 1u, abort_flag, status);
                    if (ok) {
                        uint32_t fb = a_smem_u32(&bar_full[s]);
                        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(fb), "r"(2 * TILE) : "memory");
                        int row = (int)((((long long)p.pool_layer * p.n_pages + page) * p.hkv + kvh) * 16);
                        uint32_t dk = sm0 + s * 2 * TILE, dv = dk + TILE;
                        // one copy per tensor: the page maps carry the head dimension's 64-element halves as a third
                        // dimension, so the box covers the whole K (or V) page of this KV head
                        asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
                                     ::"r"(dk), "l"(&tmK), "r"(0), "r"(row), "r"(0), "r"(fb) : "memory");
                        asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
                                     ::"r"(dv), "l"(&tmV), "r"(0), "r"(row), "r"(0), "r"(fb) : "memory");
                    }
                }
                ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
                if (!ok) { i0 = n_pg; break; }
            }
        }
    } else {
        // ---- consumers: warp w owns stacked rows mg * kAttnGroupRows + w*16 .. +15
        const int r_lo = mg * kAttnGroupRows + warp * 16 + (lane >> 2), r_hi = r_lo + 8;
        const int j_lo = r_lo / p.G, g_lo = r_lo % p.G, j_hi = r_hi / p.G, g_hi = r_hi % p.G;
        const bool v_lo = r_lo < QR && j_lo < nr, v_hi = r_hi < QR && j_hi < nr;
        const int kmax_lo = v_lo ? p0 + j_lo : -1, kmax_hi = v_hi ? p0 + j_hi : -1;
        const int nq = p.hq * HD;
        const float *q_lo = p.q + ((size_t)(b * a.R_pad + j_lo) * nq + (size_t)(kvh * p.G + g_lo) * HD);
        const float *q_hi = p.q + ((size_t)(b * a.R_pad + j_hi) * nq + (size_t)(kvh * p.G + g_hi) * HD);
        uint32_t qh[KS][4], ql[KS][4];
        const int c2 = (lane & 3) * 2;
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
#pragma unroll
            for (int part = 0; part < 4; ++part) {   // a0: (lo, cols), a1: (hi, cols), a2: (lo, cols+8), a3: (hi, cols+8)
                const bool hi_row = part & 1;
                const float *src = hi_row ? q_hi : q_lo;
                const bool valid = hi_row ? v_hi : v_lo;
                int col = ks * 16 + c2 + ((part & 2) ? 8 : 0);
                float x0 = 0.f, x1 = 0.f;
                if (valid) { float2 t = *reinterpret_cast<const float2 *>(src + col); x0 = t.x * p.scale_log2; x1 = t.y * p.scale_log2; }
                float h0 = __bfloat162float(__float2bfloat16_rn(x0)), h1 = __bfloat162float(__float2bfloat16_rn(x1));
                qh[ks][part] = pack_bf16(x0, x1);
                ql[ks][part] = pack_bf16(x0 - h0, x1 - h1);
            }
        }
        float o[NT][4];
#pragma unroll
        for (int n = 0; n < NT; ++n) { o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f; }
        float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;
        bool ok = true;
        for (int i = 0; i < n_pg && ok; ++i) {
            const int s = i % kAttnStages;
            const uint32_t ph = (uint32_t)(i / kAttnStages) & 1u;
            ok = a_wait(a_smem_u32(&bar_full[s]), ph, abort_flag, status);
            if (!ok) break;
            const uint32_t sk = sm0 + s * 2 * TILE, sv = sk + TILE;
            float sc[2][4];
#pragma unroll
            for (int n = 0; n < 2; ++n) sc[n][0] = sc[n][1] = sc[n][2] = sc[n][3] = 0.f;
            const int mat = lane >> 3, rin = lane & 7;
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) {
                int key = (mat >> 1) * 8 + rin;
                int chunk16 = (ks & 3) * 2 + (mat & 1);
                uint32_t addr = sk + (ks >> 2) * 2048 + key * 128 + ((chunk16 ^ (key & 7)) << 4);
                uint32_t kb[4];
                ldmatrix_x4(addr, kb);
                mma_bf16_16816(sc[0], qh[ks], kb[0], kb[1]);
                mma_bf16_16816(sc[0], ql[ks], kb[0], kb[1]);
                mma_bf16_16816(sc[1], qh[ks], kb[2], kb[3]);
                mma_bf16_16816(sc[1], ql[ks], kb[2], kb[3]);
            }
            // causal / validity mask and online softmax (scores are already in log2 units)
            const int key0 = (pg0 + i) * 16;
            float mx_lo = -INFINITY, mx_hi = -INFINITY;
#pragma unroll
            for (int n = 0; n < 2; ++n)
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    int key = key0 + n * 8 + c2 + e;
                    if (key > kmax_lo) sc[n][e] = -INFINITY;
                    if (key > kmax_hi) sc[n][2 + e] = -INFINITY;
                    mx_lo = fmaxf(mx_lo, sc[n][e]);
                    mx_hi = fmaxf(mx_hi, sc[n][2 + e]);
                }
            mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 1));
            mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 2));
            mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 1));
            mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 2));
            const float mn_lo = fmaxf(m_lo, mx_lo), mn_hi = fmaxf(m_hi, mx_hi);
            const float base_lo = (mn_lo == -INFINITY) ? 0.f : mn_lo, base_hi = (mn_hi == -INFINITY) ? 0.f : mn_hi;
            const float cr_lo = exp2f(m_lo - base_lo), cr_hi = exp2f(m_hi - base_hi);
            m_lo = mn_lo; m_hi = mn_hi;
            uint32_t pa[4];
            float ps_lo = 0.f, ps_hi = 0.f;
            {
                float e00 = exp2f(sc[0][0] - base_lo), e01 = exp2f(sc[0][1] - base_lo);
                float e02 = exp2f(sc[0][2] - base_hi), e03 = exp2f(sc[0][3] - base_hi);
                float e10 = exp2f(sc[1][0] - base_lo), e11 = exp2f(sc[1][1] - base_lo);
                float e12 = exp2f(sc[1][2] - base_hi), e13 = exp2f(sc[1][3] - base_hi);
                ps_lo = e00 + e01 + e10 + e11;
                ps_hi = e02 + e03 + e12 + e13;
                pa[0] = pack_bf16(e00, e01); pa[1] = pack_bf16(e02, e03);
                pa[2] = pack_bf16(e10, e11); pa[3] = pack_bf16(e12, e13);
            }
            l_lo = l_lo * cr_lo + ps_lo;
            l_hi = l_hi * cr_hi + ps_hi;
#pragma unroll
            for (int n = 0; n < NT; ++n) { o[n][0] *= cr_lo; o[n][1] *= cr_lo; o[n][2] *= cr_hi; o[n][3] *= cr_hi; }
#pragma unroll
            for (int n = 0; n < NT; n += 2) {
                int key = (mat & 1) * 8 + rin;
                int cg = n + (mat >> 1);          // 16-byte column block of V (8 dims)
                uint32_t addr = sv + (cg >> 3) * 2048 + key * 128 + (((cg & 7) ^ (key & 7)) << 4);
                uint32_t vb[4];
                ldmatrix_x4_trans(addr, vb);
                mma_bf16_16816(o[n], pa, vb[0], vb[1]);
                mma_bf16_16816(o[n + 1], pa, vb[2], vb[3]);
            }
            __syncwarp();
            if (lane == 0)
                asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(a_smem_u32(&bar_empty[s])) : "memory");
        }
        // ---- split record: unnormalised O, running max (log2 units), running sum
        l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1);
        l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
        l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1);
        l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);
        if (!ok) { l_lo = l_hi = 0.f; m_lo = m_hi = -INFINITY; }
        if (v_lo) {
            float *dst = p.part + ((((size_t)(b * a.R_pad + j_lo) * p.hq + kvh * p.G + g_lo) * p.n_splits + split) * (HD + 2));
#pragma unroll
            for (int n = 0; n < NT; ++n) *reinterpret_cast<float2 *>(dst + n * 8 + c2) = make_float2(o[n][0], o[n][1]);
            if ((lane & 3) == 0) { dst[HD] = m_lo; dst[HD + 1] = l_lo; }
        }
        if (v_hi) {
            float *dst = p.part + ((((size_t)(b * a.R_pad + j_hi) * p.hq + kvh * p.G + g_hi) * p.n_splits + split) * (HD + 2));
#pragma unroll
            for (int n = 0; n < NT; ++n) *reinterpret_cast<float2 *>(dst + n * 8 + c2) = make_float2(o[n][2], o[n][3]);
            if ((lane & 3) == 0) { dst[HD] = m_hi; dst[HD + 1] = l_hi; }
        }
    }
    __syncthreads();
    if (s_abort && threadIdx.x == 0) {  // let copies in flight land before the shared memory is released
        for (int s = 0; s < kAttnStages; ++s)
            for (uint32_t it = 0; it < (1u << 16); ++it)
                if (a_try_wait(a_smem_u32(&bar_full[s]), 0) || a_try_wait(a_smem_u32(&bar_full[s]), 1)) break;
    }
}

// Combine the split records of every (row, q head) in split order and write the attention output
// as bf16 hi / lo planes for the O projection.  One warp per (row, head).
template <int HD>
__global__ void attention_merge_kernel(StageArgs a, RowMeta rm, const float *part, int n_splits, int hq,
                                       __nv_bfloat16 *out, int T_alloc, int plain) {
    pdl_launch_dependents();
    pdl_wait();
    constexpr int E = HD / 32;
    int gw = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    int t = gw / hq, h = gw % hq;
    if (t >= a.batch * a.R_pad) return;
    int b = t / a.R_pad, j = t % a.R_pad;
    int nq = hq * HD;
    __nv_bfloat16 *ohi = out + (size_t)t * nq + h * HD + lane * E;
    __nv_bfloat16 *olo = out + ((size_t)T_alloc + t) * nq + h * HD + lane * E;
    float acc[E];
#pragma unroll
    for (int e = 0; e < E; ++e) acc[e] = 0.f;
    float inv = 0.f;
    if (j < rm.n_rows[b]) {
        const float *base = part + ((size_t)t * hq + h) * n_splits * (HD + 2);
        float M = -INFINITY;
        for (int s = 0; s < n_splits; ++s) M = fmaxf(M, base[(size_t)s * (HD + 2) + HD]);
        float L = 0.f;
        for (int s = 0; s < n_splits; ++s) {
            const float *r = base + (size_t)s * (HD + 2);
            float ms = r[HD], ls = r[HD + 1];
            if (ls <= 0.f || ms == -INFINITY) continue;
            float w = exp2f(ms - M);
            L += ls * w;
#pragma unroll
            for (int e = 0; e < E; ++e) acc[e] += w * r[lane * E + e];
        }
        inv = L > 0.f ? 1.0f / L : 0.f;
    }
#pragma unroll
    for (int e = 0; e < E; ++e) split_hi_lo(acc[e] * inv, ohi[e], olo[e], plain);
}

}  // namespace hispec
