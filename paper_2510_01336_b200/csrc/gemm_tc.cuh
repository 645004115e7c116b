// a2/a5/a6/a7/a9: the weight-streaming projections on the 5th-generation tensor cores.
//
// Y[t][n] = sum_k W[n][k] * X[t][k] with few activation rows (t <= 256) and many weight
// rows, so the operands are swapped: the weight tile (128 rows x 64 k, K-major, 128-byte
// swizzle, fetched by TMA) is the UMMA "A" operand (M = 128), the activation rows are the
// "B" operand (N = rows, or 2 x rows when the activations come as a bf16 hi plane and a
// bf16 lo plane), and the fp32 accumulator D[128][N] lives in tensor memory: TMEM lane =
// weight row, TMEM column = activation row.  The kernel is bound by streaming W from HBM:
// one warp keeps a ring of TMA stages full, one thread issues tcgen05.mma, four warps read
// the accumulator back with tcgen05.ld and either store split-K partial sums or, for the
// exit head, reduce each column to its top-2 logits so that logits never reach HBM.
//
// Every wait on an mbarrier is bounded; a wait that runs out sets HISPEC_ST_TIMEOUT in the
// status word and the CTA drains and exits.
#pragma once

#include "kernels.cuh"

namespace hispec {

constexpr uint32_t kSpinLimit = 1u << 24;
constexpr int kGemmThreads = 192;  // warp 0: TMA, warp 1: MMA + TMEM alloc, warps 2..5: epilogue
constexpr int kWTileBytes = kWeightTileRows * kTileK * 2;  // 16 KiB
constexpr int kGemmMaxDynSmem = 220 * 1024;                // dynamic shared memory the kernel may be given

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok;
}
__device__ __forceinline__ uint32_t mbar_test_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n .reg .pred p;\n mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok;
}
// bounded busy-poll variant (no hardware suspension between polls)
__device__ __forceinline__ bool mbar_spin(uint32_t bar, uint32_t parity, volatile int *abort_flag, uint32_t *status) {
    for (uint32_t it = 0; it < (1u << 28); ++it) {
        if (mbar_test_wait(bar, parity)) return true;
        if ((it & 65535u) == 65535u && *abort_flag) return false;
    }
    *abort_flag = 1;
    atomicOr(status, HISPEC_ST_TIMEOUT);
    return false;
}
// bounded wait; returns false (and raises the abort flag) when it gives up
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, uint32_t *status) {
    for (uint32_t it = 0; it < kSpinLimit; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 1023u) == 1023u && *abort_flag) return false;
    }
    *abort_flag = 1;
    atomicOr(status, HISPEC_ST_TIMEOUT);
    return false;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *tm, int x, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
        "l"(tm), "r"(x), "r"(y), "r"(bar)
        : "memory");
}
// weight tiles are read once: evict-first keeps them from displacing re-read data in L2
__device__ __forceinline__ void tma_load_2d_stream(uint32_t dst, const CUtensorMap *tm, int x, int y, uint32_t bar,
                                                   uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3}], [%4], %5;" ::"r"(dst),
        "l"(tm), "r"(x), "r"(y), "r"(bar), "l"(policy)
        : "memory");
}
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
    uint64_t policy;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
    return policy;
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *tm, int x, int y, int z, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];" ::"r"(dst),
        "l"(tm), "r"(x), "r"(y), "r"(z), "r"(bar)
        : "memory");
}
// K-major operand tile with 128-byte rows and 128-byte swizzle: 8-row groups 1024 B apart
__device__ __forceinline__ uint64_t umma_desc_sw128(uint32_t saddr) {
    uint64_t d = (uint64_t)((saddr & 0x3FFFFu) >> 4);
    d |= (uint64_t)1 << 16;            // leading-dimension offset: unused for swizzled K-major
    d |= (uint64_t)(1024u >> 4) << 32; // stride between 8-row groups
    d |= (uint64_t)1 << 46;            // descriptor version of this architecture
    d |= (uint64_t)2 << 61;            // 128-byte swizzle
    return d;
}
// kind::f16 instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = 128
__host__ __device__ inline uint32_t umma_idesc_bf16(int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
}
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
    asm volatile(
        "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}" ::"r"(tmem_d),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc)
        : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, float *v) {
    uint32_t r[8];
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "r"(taddr)
                 : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = __uint_as_float(r[i]);
}

struct GemmArgs {
    int N, K;            // weight rows (output features), reduction length
    int kb_total, splits;
    int row0, rows;      // activation rows [row0, row0 + rows) of the call
    int t_box, planes;   // rows per plane in the B tile (multiple of 8), 1 or 2 planes
    int split_planes;    // 2 planes with more than 128 rows: one MMA per plane (N = t_box each), lo accumulator at column 256
    int stages;
    int tmem_cols;       // power of two >= max(32, t_box * planes)
    int head;            // 0: store partial sums; 1: exit head (top-2 per column, optional logits)
    float *part;         // [splits][T_pad][N]
    size_t split_stride;
    float *top_part;     // head: [4 * tiles][T_pad][4]
    int T_pad;
    float *logits;       // head, optional: caller's [batch][max_rows][vocab]
    int R_pad, max_rows;
    const int32_t *n_rows;
    uint32_t *status;
};

__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmX, GemmArgs g) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_full[16], bar_empty[16], bar_acc;
    __shared__ uint32_t s_tmem;
    __shared__ int s_abort;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int tile = blockIdx.x, sp = blockIdx.y;
    const int kb0 = (int)((long long)g.kb_total * sp / g.splits);
    const int kb1 = (int)((long long)g.kb_total * (sp + 1) / g.splits);
    const int nkb = kb1 - kb0;
    const int ncols = g.t_box * g.planes;                 // rows of the B tile in shared memory
    const int mma_n = g.split_planes ? g.t_box : ncols;   // N of one MMA
    const int lo_col = g.split_planes ? 256 : g.t_box;    // accumulator column where the lo plane's results start
    const uint32_t x_bytes = (uint32_t)ncols * 128u;
    const uint32_t stage_bytes = kWTileBytes + x_bytes;
    const uint32_t smem0 = (smem_u32(smem_raw) + 1023u) & ~1023u;
    volatile int *abort_flag = &s_abort;

    if (threadIdx.x == 0) {
        s_abort = 0;
        for (int s = 0; s < g.stages; ++s) {
            mbar_init(smem_u32(&bar_full[s]), 1);
            mbar_init(smem_u32(&bar_empty[s]), 1);
        }
        mbar_init(smem_u32(&bar_acc), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem)),
                     "r"((uint32_t)g.tmem_cols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_d = s_tmem;
    pdl_launch_dependents();

    if (warp == 0) {
        if (lane == 0) {
            // Weights do not depend on the previous kernel: fill the ring with weight tiles
            // first, then wait for the producer of the activations.
            int pre = nkb < g.stages ? nkb : g.stages;
            const uint64_t policy = l2_policy_evict_first();
            for (int i = 0; i < pre; ++i) {
                uint32_t fb = smem_u32(&bar_full[i]);
                mbar_expect_tx(fb, stage_bytes);
                tma_load_2d_stream(smem0 + i * stage_bytes, &tmW, (kb0 + i) * kTileK, tile * kWeightTileRows, fb, policy);
            }
            pdl_wait();
            for (int i = 0; i < pre; ++i)
                tma_load_3d(smem0 + i * stage_bytes + kWTileBytes, &tmX, (kb0 + i) * kTileK, g.row0, 0,
                            smem_u32(&bar_full[i]));
            int s = pre == g.stages ? 0 : pre;   // slot and phase bit advance without divisions
            uint32_t ph = pre == g.stages ? 1u : 0u;
            for (int i = pre; i < nkb; ++i) {
                if (!mbar_wait(smem_u32(&bar_empty[s]), ph ^ 1u, abort_flag, g.status)) break;
                uint32_t fb = smem_u32(&bar_full[s]);
                mbar_expect_tx(fb, stage_bytes);
                tma_load_2d_stream(smem0 + s * stage_bytes, &tmW, (kb0 + i) * kTileK, tile * kWeightTileRows, fb, policy);
                tma_load_3d(smem0 + s * stage_bytes + kWTileBytes, &tmX, (kb0 + i) * kTileK, g.row0, 0, fb);
                if (++s == g.stages) { s = 0; ph ^= 1u; }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_bf16(mma_n);
            bool ok = true;
            int s = 0;
            uint32_t ph = 0;
            for (int i = 0; i < nkb && ok; ++i) {
                ok = mbar_wait(smem_u32(&bar_full[s]), ph, abort_flag, g.status);
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                uint64_t ad = umma_desc_sw128(smem0 + s * stage_bytes);
                uint64_t bd = umma_desc_sw128(smem0 + s * stage_bytes + kWTileBytes);
#pragma unroll
                for (int k = 0; k < kTileK / 16; ++k) {
                    umma_bf16(tmem_d, ad + (uint64_t)(2 * k), bd + (uint64_t)(2 * k), idesc, (i | k) ? 1u : 0u);
                    if (g.split_planes)   // the lo plane sits t_box rows (128 bytes each) further on in the tile
                        umma_bf16(tmem_d + 256u, ad + (uint64_t)(2 * k), bd + (uint64_t)((g.t_box * 128) >> 4) + (uint64_t)(2 * k),
                                  idesc, (i | k) ? 1u : 0u);
                }
                umma_commit(smem_u32(&bar_empty[s]));  // stage reusable once these MMAs have read it
                if (++s == g.stages) { s = 0; ph ^= 1u; }
            }
            umma_commit(smem_u32(&bar_acc));           // accumulator complete
        }
    } else {
        // epilogue warps: TMEM lanes 32*(warp%4) .. +31 are this warp's
        pdl_wait();  // partial-sum / top-2 buffers are read by the previous kernels' successors
        const int lg = warp & 3;
        bool ok = mbar_wait(smem_u32(&bar_acc), 0, abort_flag, g.status);
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const int n = tile * kWeightTileRows + lg * 32 + lane;
        const uint32_t taddr = tmem_d + ((uint32_t)(lg * 32) << 16);
        if (ok && nkb > 0) {
            for (int c0 = 0; c0 < g.rows; c0 += 8) {
                float v[8], w[8];
                tmem_ld8(taddr + (uint32_t)c0, v);
                if (g.planes == 2) {
                    tmem_ld8(taddr + (uint32_t)(lo_col + c0), w);
#pragma unroll
                    for (int i = 0; i < 8; ++i) v[i] += w[i];
                }
                if (!g.head) {
                    if (n < g.N) {
#pragma unroll
                        for (int i = 0; i < 8; ++i)
                            if (c0 + i < g.rows)
                                g.part[sp * g.split_stride + (size_t)(g.row0 + c0 + i) * g.N + n] = v[i];
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        if (c0 + i >= g.rows) break;  // uniform across the warp
                        int t = g.row0 + c0 + i;
                        float val = (n < g.N) ? v[i] : -INFINITY;
                        if (g.logits && n < g.N) {
                            int b = t / g.R_pad, j = t % g.R_pad;
                            if (j < g.n_rows[b]) g.logits[((size_t)b * g.max_rows + j) * g.N + n] = val;
                        }
                        Top2 best = top2_warp(Top2{val, -INFINITY, n < g.N ? n : 0x7fffffff});
                        if (lane == 0) {
                            float *o = g.top_part + ((size_t)(tile * 4 + lg) * g.T_pad + t) * 4;
                            o[0] = best.v1;
                            o[1] = __int_as_float(best.i1);
                            o[2] = best.v2;
                        }
                    }
                }
            }
        } else if (ok && !g.head) {  // empty split: contributes zeros
            if (n < g.N)
                for (int c = 0; c < g.rows; ++c) g.part[sp * g.split_stride + (size_t)(g.row0 + c) * g.N + n] = 0.0f;
        }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    }
    __syncthreads();
    if (s_abort && threadIdx.x == 0) {
        // give copies that are still in flight a bounded chance to land before the CTA's
        // shared memory goes away
        for (int s = 0; s < g.stages && s < nkb; ++s)
            for (uint32_t it = 0; it < (1u << 16); ++it)
                if (mbar_try_wait(smem_u32(&bar_full[s]), 0) || mbar_try_wait(smem_u32(&bar_full[s]), 1)) break;
    }
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_d), "r"((uint32_t)g.tmem_cols)
                     : "memory");
    }
}


// ---- the same projection for many rows (more than 64): two weight tiles per CTA share one activation tile ------
// With T rows the activation tile of a k-block is T x 128 bytes per plane -- larger than the 16 KiB weight tile from
// 64 rows on -- and it is re-read for every weight tile.  Here a CTA takes TWO adjacent weight tiles (256 output
// features) per activation tile, which halves that traffic and leaves room for a deeper ring of weight blocks (one
// CTA per SM, all of its shared memory).  Both planes of the activations accumulate into the SAME accumulator
// (W.hi + W.lo is what the epilogue would add anyway), so an accumulator has t_box <= 256 columns: tile 0 at
// column 0, tile 1 at column 256.
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_pair_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmX, GemmArgs g) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_full[16], bar_empty[16], bar_acc;
    __shared__ uint32_t s_tmem;
    __shared__ int s_abort;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int pair = blockIdx.x, sp = blockIdx.y;
    const int tile0 = 2 * pair;
    const bool two = (tile0 + 1) * kWeightTileRows < g.N;   // the second tile exists
    const int kb0 = (int)((long long)g.kb_total * sp / g.splits);
    const int kb1 = (int)((long long)g.kb_total * (sp + 1) / g.splits);
    const int nkb = kb1 - kb0;
    const uint32_t x_bytes = (uint32_t)(g.t_box * g.planes) * 128u;
    const uint32_t w_bytes = two ? 2u * kWTileBytes : kWTileBytes;
    const uint32_t stage_bytes = 2u * kWTileBytes + x_bytes;
    const uint32_t smem0 = (smem_u32(smem_raw) + 1023u) & ~1023u;
    volatile int *abort_flag = &s_abort;

    if (threadIdx.x == 0) {
        s_abort = 0;
        for (int s = 0; s < g.stages; ++s) {
            mbar_init(smem_u32(&bar_full[s]), 1);
            mbar_init(smem_u32(&bar_empty[s]), 1);
        }
        mbar_init(smem_u32(&bar_acc), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem)), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_d = s_tmem;
    pdl_launch_dependents();

    if (warp == 0) {
        if (lane == 0) {
            const uint64_t policy = l2_policy_evict_first();
            auto load_w = [&](int s, int kb) {
                const uint32_t fb = smem_u32(&bar_full[s]);
                mbar_expect_tx(fb, w_bytes + x_bytes);
                tma_load_2d_stream(smem0 + s * stage_bytes, &tmW, kb * kTileK, tile0 * kWeightTileRows, fb, policy);
                if (two)
                    tma_load_2d_stream(smem0 + s * stage_bytes + kWTileBytes, &tmW, kb * kTileK, (tile0 + 1) * kWeightTileRows, fb,
                                       policy);
            };
            // weights do not depend on the previous kernel: fill the ring with them first
            const int pre = nkb < g.stages ? nkb : g.stages;
            for (int i = 0; i < pre; ++i) load_w(i, kb0 + i);
            pdl_wait();
            for (int i = 0; i < pre; ++i)
                tma_load_3d(smem0 + i * stage_bytes + 2 * kWTileBytes, &tmX, (kb0 + i) * kTileK, g.row0, 0, smem_u32(&bar_full[i]));
            int s = pre == g.stages ? 0 : pre;
            uint32_t ph = pre == g.stages ? 1u : 0u;
            for (int i = pre; i < nkb; ++i) {
                if (!mbar_wait(smem_u32(&bar_empty[s]), ph ^ 1u, abort_flag, g.status)) break;
                load_w(s, kb0 + i);
                tma_load_3d(smem0 + s * stage_bytes + 2 * kWTileBytes, &tmX, (kb0 + i) * kTileK, g.row0, 0, smem_u32(&bar_full[s]));
                if (++s == g.stages) { s = 0; ph ^= 1u; }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_bf16(g.t_box);
            const uint64_t lo_off = (uint64_t)((g.t_box * 128) >> 4);   // the lo plane sits t_box rows further on
            bool ok = true;
            int s = 0;
            uint32_t ph = 0;
            for (int i = 0; i < nkb && ok; ++i) {
                ok = mbar_wait(smem_u32(&bar_full[s]), ph, abort_flag, g.status);
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint64_t a0 = umma_desc_sw128(smem0 + s * stage_bytes);
                const uint64_t a1 = umma_desc_sw128(smem0 + s * stage_bytes + kWTileBytes);
                const uint64_t bd = umma_desc_sw128(smem0 + s * stage_bytes + 2 * kWTileBytes);
#pragma unroll
                for (int k = 0; k < kTileK / 16; ++k) {
                    const uint64_t kk = (uint64_t)(2 * k);
                    umma_bf16(tmem_d, a0 + kk, bd + kk, idesc, (i | k) ? 1u : 0u);
                    if (g.planes == 2) umma_bf16(tmem_d, a0 + kk, bd + lo_off + kk, idesc, 1u);
                    if (two) {
                        umma_bf16(tmem_d + 256u, a1 + kk, bd + kk, idesc, (i | k) ? 1u : 0u);
                        if (g.planes == 2) umma_bf16(tmem_d + 256u, a1 + kk, bd + lo_off + kk, idesc, 1u);
                    }
                }
                umma_commit(smem_u32(&bar_empty[s]));
                if (++s == g.stages) { s = 0; ph ^= 1u; }
            }
            umma_commit(smem_u32(&bar_acc));
        }
    } else {
        pdl_wait();
        const int lg = warp & 3;
        const bool ok = mbar_wait(smem_u32(&bar_acc), 0, abort_flag, g.status);
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        for (int t2 = 0; t2 < (two ? 2 : 1); ++t2) {
            const int tile = tile0 + t2;
            const int n = tile * kWeightTileRows + lg * 32 + lane;
            const uint32_t taddr = tmem_d + (uint32_t)(256 * t2) + ((uint32_t)(lg * 32) << 16);
            if (ok && nkb > 0) {
                for (int c0 = 0; c0 < g.rows; c0 += 8) {
                    float v[8];
                    tmem_ld8(taddr + (uint32_t)c0, v);
                    if (!g.head) {
                        if (n < g.N) {
#pragma unroll
                            for (int i = 0; i < 8; ++i)
                                if (c0 + i < g.rows) g.part[sp * g.split_stride + (size_t)(g.row0 + c0 + i) * g.N + n] = v[i];
                        }
                    } else {
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            if (c0 + i >= g.rows) break;   // uniform across the warp
                            const int t = g.row0 + c0 + i;
                            const float val = (n < g.N) ? v[i] : -INFINITY;
                            if (g.logits && n < g.N) {
                                const int b = t / g.R_pad, j = t % g.R_pad;
                                if (j < g.n_rows[b]) g.logits[((size_t)b * g.max_rows + j) * g.N + n] = val;
                            }
                            const Top2 best = top2_warp(Top2{val, -INFINITY, n < g.N ? n : 0x7fffffff});
                            if (lane == 0) {
                                float *o = g.top_part + ((size_t)(tile * 4 + lg) * g.T_pad + t) * 4;
                                o[0] = best.v1; o[1] = __int_as_float(best.i1); o[2] = best.v2;
                            }
                        }
                    }
                }
            } else if (ok && !g.head) {   // empty split: contributes zeros
                if (n < g.N)
                    for (int c = 0; c < g.rows; ++c) g.part[sp * g.split_stride + (size_t)(g.row0 + c) * g.N + n] = 0.0f;
            }
        }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    }
    __syncthreads();
    if (s_abort && threadIdx.x == 0) {
        for (int s = 0; s < g.stages && s < nkb; ++s)
            for (uint32_t it = 0; it < (1u << 16); ++it)
                if (mbar_try_wait(smem_u32(&bar_full[s]), 0) || mbar_try_wait(smem_u32(&bar_full[s]), 1)) break;
    }
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_d), "r"(512u) : "memory");
    }
}

}  // namespace hispec
