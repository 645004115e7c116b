// One persistent kernel per stage call: every step a0..a10 of the call runs inside a single
// cooperative launch with one CTA per SM.
//
// Why: at batch 1 a call is ~80 dependent kernels of 5-50 us each, and every kernel boundary
// drains the HBM pipe for several microseconds.  Here the weights -- which depend on nothing
// the call computes -- are streamed by a dedicated TMA warp that runs through the *whole*
// call's schedule of weight tiles, limited only by free slots in a deep shared-memory ring, so
// HBM keeps flowing across the dependency points (grid barriers, attention, element-wise
// phases).  The other warps work phase by phase:
//
//   projection phase   two independent pipelines per CTA (measured: one TMA ring + one MMA thread
//                      per SM tops out near 4.9 TB/s, two reach the HBM limit): warp 0
//                      streams weights, warps 1/2 issue tcgen05.mma (accumulators in TMEM,
//                      double buffered per pipeline), warp 3 TMA-loads the activation
//                      operand, warps 4-7 drain TMEM to split-K partial sums (stream-K partition over 2 x grid
//                      "virtual CTAs": every pipeline gets the same number of 128x64 weight
//                      blocks, +-1), or, for the exit head, to top-2 records (there the two
//                      pipelines take the two halves of each tile's K range);
//   element-wise phase warps 1-7 of all CTAs: sum the partial slots in slot order, then
//                      RoPE + KV append / residual + gain + hi-lo split / SiLU*up / split merge;
//   attention phase    warp 3 stages KV pages by TMA, warps 4-7 run the tiled attention;
//   final phase        CTA b reduces sequence b's top-2 records and applies LeadingSubstringVerify.
//
// RMSNorm is applied as y = W (g .* x) / rms(x): the projection runs on g .* x and the row's
// 1/rms (from per-chunk sums of squares written by the producing phase) scales the result where
// the partial sums are consumed, so no grid barrier is needed between "residual" and "norm".
//
// Phases are separated by a grid barrier (counter + generation word in global memory).  Every
// wait -- mbarrier or grid barrier -- is bounded; on a timeout the CTA raises an abort flag,
// sets HISPEC_ST_TIMEOUT, and all later waits fall through so that the kernel drains and exits.
#pragma once
#include <type_traits>

#include "attention.cuh"
#include "gemm_tc.cuh"

namespace hispec {

// Eight warps, two per scheduler partition: with ten, a partition with three warps limits every thread to
// 168 registers, and the spills that caused cost every phase a memory round trip.
constexpr int kMegaThreads = 256;
constexpr int kMegaMaxStages = 8;  // per pipeline
constexpr int kMegaAttnStages = 16; // most KV pages in flight per CTA in the attention phase (8 KB each at head_dim 128); a call uses 4 to 16
constexpr int kMegaMaxBatch = 64;
constexpr int kMegaWorkers = 224;  // threads of warps 1..7
constexpr int kMegaLeader = 32;    // warp 1 lane 0
// warp 0: one thread streams the weights of both pipelines; warps 1/2: tcgen05.mma of pipelines 0/1; warp 3:
// activation operand of both pipelines and attention pages; warps 4..7: accumulator drain / attention tiles.
// Warps 1..7 are the workers of the element-wise phases.
constexpr int kWarpMma0 = 1, kWarpX = 3, kWarpEpi0 = 4;
constexpr int kMegaAccCols = 128;  // TMEM columns per accumulator buffer (2 pipelines x 2 buffers)
constexpr int kEwChunk = 256;      // columns per element-wise work item (one warp, 8 per lane)
constexpr int kSsqChunk = 128;     // columns per sum-of-squares record
constexpr int kMegaMaxDynSmem = 212 * 1024;   // dynamic shared memory of the kernel: 227 KB per CTA less its static tables
constexpr int kMegaSlotTiles = 512; // output tiles per projection whose partial-slot ranges are tabulated in shared memory

struct __align__(64) MegaGemm {
    CUtensorMap tmW;
    int N, K, tiles, kb_total;
    int pad[12];
};

struct MegaArgs {
    StageArgs a;
    const MegaGemm *gemms;  // [n_layers][4]: QKV, O, gate/up, down
    const MegaGemm *head;
    const float *const *attn_norm;
    const float *const *ffn_norm;
    const float *final_norm;
    int d, hq, hkv, hd, ffn, vocab;
    float eps;
    int T_pad, T_alloc, t_box, planes, stages, plain;
    int32_t *len_d, *len_i, *len_f;
    const int32_t *n_rows_in, *n_draft_in, *tokens, *n_tokens;
    const __nv_bfloat16 *tok_emb;
    const float *h_src;
    float *exit_buf, *hidden_out;
    __nv_bfloat16 *k_pages, *v_pages;
    const int32_t *block_table;
    long long n_pages;
    int first_layer;
    float *x;
    __nv_bfloat16 *act_d, *act_o, *act_f;
    float *q, *part, *attn_part, *top_part, *ssq;
    // a block of draft steps in one launch (hispec_draft_block): the call's steps a0..a10 run n_rep times; step s > 0
    // reads its token from block[b * block_stride + s - 1], step s < n_steps writes block[b * block_stride + s]
    int attn_log2;           // attn_stages == 1 << attn_log2
    int attn_stages;         // KV pages in flight per CTA (4 at short contexts: 8 measured +2 % on a 12-row call at context 1024, -2 % at 16384)
    int attn_in_ring;        // where the attention phase stages its KV pages: 0 an area of its own behind the rings, 1 the activation
                             // areas of the ring stages, 2 the whole of both rings (the weight producer then holds the output
                             // projection's blocks back until the CTA's attention items are done)
    int n_rep, n_steps, block_stride;
    int32_t *block;
    float *cta_top;          // [gridDim.x][T_pad][4]: each CTA's top-2 over its own exit-head tiles (v1, id1, v2, -)
    const double *inv_freq;
    float2 *rope;            // [T_pad][hd / 2] (cos, sin) of each row's position, filled in the first phase
    int n_splits, n_mg, mt, G;
    int ngrp;                // warp groups that share an attention item's pages (4, 2 or 1); records per (row, head) = n_splits * ngrp
    float scale_log2;
    AcceptArgs r;
    int32_t *argmax_ws;
    float *logits;
    uint32_t *status;
    unsigned *bar_count;     // this launch's barrier counter (zero at launch)
    unsigned *bar_next;      // the next launch's counter: zeroed by this launch
    unsigned long long *trace;  // optional: CTA 0 stamps the global timer after every grid barrier
};

// Segment lists (tile, k-block range) of this CTA's two pipelines for each kind of projection, worked out
// once at kernel start: the role loops are single threads, for which a 64-bit division costs about a
// microsecond of pure latency.
constexpr int kMegaMaxSegs = 16;
struct SegList {
    int n;
    int tile[kMegaMaxSegs];
    short kb0[kMegaMaxSegs], kb1[kMegaMaxSegs];
};

struct MegaShared {
    SegList segs[5][2];      // [QKV, O, gate/up, down, head][pipeline]
    uint64_t w_full[2][kMegaMaxStages], x_full[2][kMegaMaxStages], empty[2][kMegaMaxStages];
    uint64_t acc_full[2][2], acc_empty[2][2];
    uint64_t a_full[kMegaAttnStages], a_empty[kMegaAttnStages];
    uint32_t tmem;
    int abort_flag;
    int attn_epoch;          // attention phases this CTA has finished (attn_in_ring == 2: releases the weight producer)
    int trace_n;
    int bar_k;
    // per output tile of the four layer projections: number of partial slots and the first pipeline that holds one
    // (worked out once: two divisions per look-up otherwise, in front of every element-wise item's loads)
    unsigned short slot_n[4][kMegaSlotTiles];
    unsigned short slot_first[4][kMegaSlotTiles];
    int stamp_on, stamp_n;   // HISPEC_STAMPS builds only: fine-grained time stamps of one layer
    int p0[kMegaMaxBatch], nr[kMegaMaxBatch], nd[kMegaMaxBatch], dst[kMegaMaxBatch];
    float red_v1[8], red_v2[8];
    int red_i1[8];
};

// token input / output of embedding-mode step `step` (a plain call has one step and block == nullptr)
__device__ __forceinline__ int mega_tok_in(const MegaArgs &m, int step, int b, int j) {
    if (step == 0 || !m.block) return m.tokens[b * m.a.tok_stride + m.a.tok_offset + j];
    return m.block[(size_t)b * m.block_stride + step - 1];
}

// Development aid (compiled with -DHISPEC_STAMPS only): lane 0 of any warp of one CTA records
// (tag * 100 + warp, global timer) pairs into the trace buffer, words 200.., while sh.stamp_on is set.
#ifdef HISPEC_STAMPS
#ifndef HISPEC_STAMP_CTA
#define HISPEC_STAMP_CTA 0
#endif
#define MEGA_STAMP(tag)                                                                                   \
    do {                                                                                                  \
        if (m.trace && blockIdx.x == HISPEC_STAMP_CTA && (threadIdx.x & 31) == 0 &&                       \
            *((volatile int *)&sh.stamp_on)) {                                                            \
            unsigned long long t_;                                                                        \
            asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t_));                                         \
            const int i_ = atomicAdd(&sh.stamp_n, 1);                                                     \
            if (i_ < 200) { m.trace[200 + 2 * i_] = (tag) * 100 + (threadIdx.x >> 5); m.trace[201 + 2 * i_] = t_; } \
        }                                                                                                 \
    } while (0)
#else
#define MEGA_STAMP(tag) do { } while (0)
#endif

// ---- stream-K partition ----------------------------------------------------------------------
// The k-blocks of a projection, numbered tile-major, are cut into gridDim.x equal spans.
__host__ __device__ inline int mega_eff_ctas(long long U, int G) { return U < (long long)G ? (int)U : G; }
__host__ __device__ inline int mega_cta_of(long long u, long long U, int G) {
    return (int)(((u + 1) * G + U - 1) / U) - 1;
}
// Pipeline p of CTA c is virtual CTA 2c + p of 2G.  In `whole` mode (exit head: the epilogue needs a
// tile's complete K range) tiles are dealt to real CTAs and pipeline p takes half p of each tile's K range.
struct SegIter {
    long long u, hi;
    int kbt, whole, p;
    __device__ SegIter(int tiles, int kb_total, int whole_, int c, int p_, int G) : kbt(kb_total), whole(whole_), p(p_) {
        if (whole) {
            u = (long long)c * tiles / G;        // tile index range
            hi = (long long)(c + 1) * tiles / G;
        } else {
            long long U = (long long)tiles * kb_total;
            int Ge = mega_eff_ctas(U, 2 * G);    // with fewer k-blocks than pipelines only the first U take part
            int vc = 2 * c + p;
            if (vc >= Ge) { u = hi = 0; return; }
            u = (long long)vc * U / Ge;
            hi = (long long)(vc + 1) * U / Ge;
        }
    }
    __device__ bool next(int &tile, int &kb0, int &kb1) {
        if (u >= hi) return false;
        if (whole) {
            tile = (int)u;
            kb0 = p ? kbt / 2 : 0;
            kb1 = p ? kbt : kbt / 2;
            ++u;
            return true;
        }
        tile = (int)(u / kbt);
        kb0 = (int)(u % kbt);
        long long rem = hi - u;
        kb1 = (rem < (long long)(kbt - kb0)) ? kb0 + (int)rem : kbt;
        u += kb1 - kb0;
        return true;
    }
};
// slots of a tile: one per CTA whose span touches it, in CTA order
__host__ __device__ inline void mega_slots(int tile, int tiles, int kbt, int G, int &first_cta, int &n_slots) {
    // 32-bit arithmetic: the host only takes this path when tiles * kbt * 2G < 2^31
    const unsigned U = (unsigned)tiles * (unsigned)kbt;
    const unsigned Ge = U < 2u * (unsigned)G ? U : 2u * (unsigned)G;
    const unsigned u0 = (unsigned)tile * (unsigned)kbt, u1 = u0 + (unsigned)kbt - 1u;
    first_cta = (int)(((u0 + 1u) * Ge + U - 1u) / U) - 1;
    n_slots = (int)(((u1 + 1u) * Ge + U - 1u) / U) - 1 - first_cta + 1;
}

// Quotient of two small non-negative integers (x < 2^21, d >= 1) through the reciprocal unit: the index arithmetic of a
// work item sits in front of its loads, on the critical path of every latency-bound phase, and a 32-bit integer
// division by a run-time value is a chain of ~30 dependent instructions.  (x + 0.5) / d is at least 0.5 / d away from
// an integer, the approximate division is off by at most 2 ulp, so truncation gives the exact quotient.
__device__ __forceinline__ int qdiv(int x, int d) { return __float2int_rz(__fdividef((float)x + 0.5f, (float)d)); }

// ---- barriers --------------------------------------------------------------------------------
__device__ __forceinline__ void worker_bar() { asm volatile("bar.sync 1, %0;" ::"n"(kMegaWorkers) : "memory"); }

__device__ __forceinline__ unsigned ld_acquire_u32(const unsigned *p) {
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
// All worker threads of all CTAs.  Global writes made before it are visible after it, also to TMA
// reads.  The counter only grows during a launch: barrier number k is passed once it has reached
// (k + 1) * gridDim.x.  Arrival is a fire-and-forget release reduction; waiting polls with acquire loads.
// `to_tma`: the phase wrote something that a later TMA load reads (activation planes, K/V pages).
__device__ __forceinline__ void grid_sync(const MegaArgs &m, MegaShared &sh, bool to_tma = true) {
    if (to_tma) asm volatile("fence.proxy.async;" ::: "memory");
    worker_bar();
    if (threadIdx.x == kMegaLeader) {
        volatile int *ab = &sh.abort_flag;
        const unsigned target = (unsigned)(++sh.bar_k) * gridDim.x;
        if (!*ab) {
            MEGA_STAMP(60);
            asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(m.bar_count) : "memory");
            bool ok = false;
            for (uint32_t it = 0; it < (1u << 26); ++it) {
                if ((int)(ld_acquire_u32(m.bar_count) - target) >= 0) { ok = true; break; }
                if ((it & 4095u) == 4095u && (*((volatile uint32_t *)m.status) & HISPEC_ST_TIMEOUT)) break;
            }
            if (!ok) {
                *ab = 1;
                atomicOr(m.status, HISPEC_ST_TIMEOUT);
            }
        }
        MEGA_STAMP(61);
        if (m.trace && blockIdx.x == 0) {
            unsigned long long t;
            asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
            int i = sh.trace_n++;
            if (i < 1000) m.trace[i] = t;
        }
    }
    worker_bar();
}

// ---- row bookkeeping (every CTA computes the same table; CTA 0 reports) -------------------------
__device__ __forceinline__ void mega_prep_rows(const MegaArgs &m, MegaShared &sh, int step, int tid, int nthreads) {
    const StageArgs &a = m.a;
    for (int b = tid; b < a.batch; b += nthreads) {
        int gA = m.len_d[b], gB = m.len_i[b], gC = m.len_f[b];
        int p0 = a.l0 < a.L_d ? gA : (a.l0 < a.L_i ? gB : gC);
        uint32_t st = 0;
        int nr, nd = 0;
        if (a.mode == 0) {
            if (m.n_tokens) {
                nr = m.n_tokens[b] - a.tok_offset;
                nr = nr < 0 ? 0 : (nr > a.R_pad ? a.R_pad : nr);
            } else {
                nr = a.fixed_rows;
                if (mega_tok_in(m, step, b, 0) < 0) nr = 0;
            }
        } else if (m.n_rows_in) {
            nr = m.n_rows_in[b];
            nd = m.n_draft_in[b];
            if (nr < 0 || nr > a.R_pad || nd < 0 || nd > nr || nr > nd + 1 || nd > a.k) { st |= HISPEC_ST_STATE; nr = 0; nd = 0; }
        } else {
            int avail = (a.l0 == a.L_d) ? gA - gB : gB - gC;
            if (avail < 0) avail = 0;
            if (a.is_target && avail > a.k) st |= HISPEC_ST_STATE;
            nr = avail < a.R_pad ? avail : a.R_pad;
            nd = nr < a.k ? nr : a.k;
        }
        if (a.l0 < a.L_d && a.l1 > a.L_d && gB != p0) st |= HISPEC_ST_STATE;
        if (a.l0 < a.L_i && a.l1 > a.L_i && gC != p0) st |= HISPEC_ST_STATE;
        if (gC > gB || gB > gA) st |= HISPEC_ST_STATE;
        if (a.mode == 1) {
            int avail = (a.l0 == a.L_d) ? gA - gB : gB - gC;
            if (avail < nr) st |= HISPEC_ST_STATE;
        }
        int dst = (a.l1 == a.L_d) ? p0 - gB : ((a.l1 == a.L_i) ? p0 - gC : 0);
        if (a.l1 != a.L_f && (dst < 0 || dst + nr > a.max_rows)) st |= HISPEC_ST_BOUNDS;
        if ((long long)p0 + nr > (long long)a.max_pages * a.page_size || p0 < 0) st |= HISPEC_ST_BOUNDS;
        if (st) {
            if (blockIdx.x == 0) atomicOr(m.status, st);
            nr = 0;
            nd = 0;
        }
        sh.p0[b] = p0; sh.nr[b] = nr; sh.nd[b] = nd; sh.dst[b] = dst;
    }
}

// 1 / rms of row t from the per-chunk sums of squares of the phase that produced the row
__device__ __forceinline__ float mega_inv_rms(const MegaArgs &m, int t) {
    const int nch = (m.d + kSsqChunk - 1) / kSsqChunk;
    float s = 0.f;
    for (int c = 0; c < nch; ++c) s += m.ssq[(size_t)t * nch + c];
    return rsqrtf(s / (float)m.d + m.eps);
}

__device__ __forceinline__ void store8_hilo(__nv_bfloat16 *hi, __nv_bfloat16 *lo, const float *v, int plain) {
    uint32_t h[4], l[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        __nv_bfloat16 h0, l0, h1, l1;
        split_hi_lo(v[2 * i], h0, l0, plain);
        split_hi_lo(v[2 * i + 1], h1, l1, plain);
        __nv_bfloat162 hh = __halves2bfloat162(h0, h1), ll = __halves2bfloat162(l0, l1);
        h[i] = *reinterpret_cast<uint32_t *>(&hh);
        l[i] = *reinterpret_cast<uint32_t *>(&ll);
    }
    *reinterpret_cast<uint4 *>(hi) = make_uint4(h[0], h[1], h[2], h[3]);
    *reinterpret_cast<uint4 *>(lo) = make_uint4(l[0], l[1], l[2], l[3]);
}

// sum of the split-K partial slots of 8 consecutive columns (all inside one tile), slot order
// part 0 / 1 of `parts` = 2 takes the first ceil(ns / 2) / the remaining slots (parts = 1: all of them)
__device__ __forceinline__ void sum_slots8(const MegaArgs &m, const MegaShared &sh, int kind, const MegaGemm &g, int t, int n,
                                           float *v, int part = 0, int parts = 1) {
    int ns = sh.slot_n[kind][n / kWeightTileRows];
    const size_t stride = (size_t)m.T_pad * g.N;
    const float *p = m.part + (size_t)t * g.N + n;
    if (parts == 2) {
        const int h0 = (ns + 1) >> 1;
        if (part) { p += (size_t)h0 * stride; ns -= h0; } else ns = h0;
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = 0.f;
    // eight slots per batch, all loads in flight together; the sum stays in slot order
    for (int s0 = 0; s0 < ns; s0 += 8) {
        float4 a[8], b[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int sidx = s0 + u < ns ? s0 + u : ns - 1;
            a[u] = *reinterpret_cast<const float4 *>(p + sidx * stride);
            b[u] = *reinterpret_cast<const float4 *>(p + sidx * stride + 4);
        }
#pragma unroll
        for (int u = 0; u < 8; ++u)
            if (s0 + u < ns) {
                v[0] += a[u].x; v[1] += a[u].y; v[2] += a[u].z; v[3] += a[u].w;
                v[4] += b[u].x; v[5] += b[u].y; v[6] += b[u].z; v[7] += b[u].w;
            }
    }
}
__device__ __forceinline__ float sum_slots1(const MegaArgs &m, const MegaShared &sh, int kind, const MegaGemm &g, int t, int n) {
    const int ns = sh.slot_n[kind][n / kWeightTileRows];
    const size_t stride = (size_t)m.T_pad * g.N;
    const float *p = m.part + (size_t)t * g.N + n;
    float v = 0.f;
    for (int s = 0; s < ns; ++s) v += p[s * stride];
    return v;
}

// ---- element-wise phases (gw: global worker-warp index, ngw: number of worker warps in the grid) ----
// a0 + gain: fetch rows, x <- row, act_d <- hi/lo(x .* gain), chunk sums of squares
__device__ void ew_rows_in(const MegaArgs &m, MegaShared &sh, const float *gain, int step, int gw, int ngw, int lane) {
    const StageArgs &a = m.a;
    const int nch = (m.d + kEwChunk - 1) / kEwChunk;
    for (int item = gw; item < m.T_pad * nch; item += ngw) {
        const int t = qdiv(item, nch), ch = item - t * nch, b = qdiv(t, a.R_pad), j = t - b * a.R_pad;
        const int c = ch * kEwChunk + lane * 8;
        bool valid = j < sh.nr[b];
        float v[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) v[i] = 0.f;
        if (valid && c < m.d) {
            if (a.mode == 0) {
                int tok = mega_tok_in(m, step, b, j);
                if (tok < 0 || tok >= m.vocab) {
                    if (lane == 0 && ch == 0) atomicOr(m.status, HISPEC_ST_BOUNDS);
                } else {
                    uint4 raw = *reinterpret_cast<const uint4 *>(m.tok_emb + (size_t)tok * m.d + c);
                    const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        v[2 * i] = __uint_as_float(w[i] << 16);
                        v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
                    }
                }
            } else {
                const float *src = m.h_src + ((size_t)b * a.max_rows + j) * m.d + c;
                float4 p = *reinterpret_cast<const float4 *>(src), q = *reinterpret_cast<const float4 *>(src + 4);
                v[0] = p.x; v[1] = p.y; v[2] = p.z; v[3] = p.w; v[4] = q.x; v[5] = q.y; v[6] = q.z; v[7] = q.w;
            }
        }
        float ss = 0.f;
        if (c < m.d) {
            float *xr = m.x + (size_t)t * m.d + c;
            *reinterpret_cast<float4 *>(xr) = make_float4(v[0], v[1], v[2], v[3]);
            *reinterpret_cast<float4 *>(xr + 4) = make_float4(v[4], v[5], v[6], v[7]);
            float gv[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) { ss += v[i] * v[i]; gv[i] = v[i] * gain[c + i]; }
            store8_hilo(m.act_d + (size_t)t * m.d + c, m.act_d + ((size_t)m.T_alloc + t) * m.d + c, gv, m.plain);
        }
        // lanes 0-15 hold the chunk's first 128 columns, lanes 16-31 the second 128: one record each
#pragma unroll
        for (int o = 8; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
        const int nrec = (m.d + kSsqChunk - 1) / kSsqChunk, rec = 2 * ch + (lane >> 4);
        if ((lane & 15) == 0 && rec < nrec) m.ssq[(size_t)t * nrec + rec] = ss;
    }
}

// (cos, sin) of every row's rotary angles, once per call (the angle is formed and reduced in fp64).
// Dealt to the grid's worker warps from the far end, so that it runs beside ew_rows_in's items.
__device__ void ew_rope_table(const MegaArgs &m, MegaShared &sh, int gw, int ngw, int lane) {
    const StageArgs &a = m.a;
    const int half = m.hd / 2;
    for (int idx = (ngw - 1 - gw) * 32 + lane; idx < m.T_pad * half; idx += ngw * 32) {
        const int t = qdiv(idx, half), i = idx - t * half, b = qdiv(t, a.R_pad), j = t - b * a.R_pad;
        double sn, cs;
        sincos((double)(sh.p0[b] + j) * m.inv_freq[i], &sn, &cs);
        m.rope[idx] = make_float2((float)cs, (float)sn);
    }
}

// a5/a7 epilogue: x += projection; act_d <- hi/lo(x .* gain); chunk sums of squares; exit rows on the last layer
__device__ void ew_resid(const MegaArgs &m, MegaShared &sh, const MegaGemm &g, int kind, const float *gain, float *exit_buf,
                         float *hidden_out, int gw, int ngw, int lane) {
    // One warp per (row, 128 columns): the half-warps each add half of the partial slots (a tile of O or
    // down has about ten), 8 columns per lane, and exchange their sums; then half 0 stores the fp32 row,
    // half 1 the bf16 operand planes.
    const StageArgs &a = m.a;
    const int nch = (m.d + kSsqChunk - 1) / kSsqChunk;
    const int hl = lane >> 4, li = lane & 15;
    for (int item = gw; item < m.T_pad * nch; item += ngw) {
        const int t = qdiv(item, nch), ch = item - t * nch, b = qdiv(t, a.R_pad), j = t - b * a.R_pad;
        const int c = ch * kSsqChunk + li * 8;
        const bool valid = j < sh.nr[b];
        float ss = 0.f;
        float v[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) v[i] = 0.f;
        float4 p = make_float4(0.f, 0.f, 0.f, 0.f), q = p, g0 = p, g1 = p;
        if (c < m.d) {
            const float *xr = m.x + (size_t)t * m.d + c;
            p = *reinterpret_cast<const float4 *>(xr);
            q = *reinterpret_cast<const float4 *>(xr + 4);
            g0 = *reinterpret_cast<const float4 *>(gain + c);   // fetched with everything else: the gain vector of a
            g1 = *reinterpret_cast<const float4 *>(gain + c + 4);   // layer is cold, one more round trip if loaded at its use
            sum_slots8(m, sh, kind, g, t, c, v, hl, 2);
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const float o = __shfl_xor_sync(0xffffffffu, v[i], 16);
            v[i] = hl ? o + v[i] : v[i] + o;   // first half + second half, the same value in both half-warps
        }
        MEGA_STAMP(76);
        if (c < m.d) {
            const float xo[8] = {p.x, p.y, p.z, p.w, q.x, q.y, q.z, q.w};
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                v[i] = valid ? v[i] + xo[i] : 0.f;
                ss += v[i] * v[i];
            }
            if (hl == 0) {
                float *xr = m.x + (size_t)t * m.d + c;
                *reinterpret_cast<float4 *>(xr) = make_float4(v[0], v[1], v[2], v[3]);
                *reinterpret_cast<float4 *>(xr + 4) = make_float4(v[4], v[5], v[6], v[7]);
                if (valid && exit_buf) {
                    float *e = exit_buf + ((size_t)b * a.max_rows + sh.dst[b] + j) * m.d + c;
                    *reinterpret_cast<float4 *>(e) = make_float4(v[0], v[1], v[2], v[3]);
                    *reinterpret_cast<float4 *>(e + 4) = make_float4(v[4], v[5], v[6], v[7]);
                }
                if (valid && hidden_out) {
                    float *e = hidden_out + ((size_t)b * a.max_rows + j) * m.d + c;
                    *reinterpret_cast<float4 *>(e) = make_float4(v[0], v[1], v[2], v[3]);
                    *reinterpret_cast<float4 *>(e + 4) = make_float4(v[4], v[5], v[6], v[7]);
                }
            } else {
                const float gn[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
                float gv[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) gv[i] = v[i] * gn[i];
                store8_hilo(m.act_d + (size_t)t * m.d + c, m.act_d + ((size_t)m.T_alloc + t) * m.d + c, gv, m.plain);
            }
        }
#pragma unroll
        for (int o = 8; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
        if (lane == 0) m.ssq[(size_t)t * nch + ch] = ss;
        MEGA_STAMP(77);
    }
}

// 1 / rms of row t in two steps, so that the caller can put its other loads between them and pay one
// memory round trip instead of two: lanes fetch the chunk sums (no use of the values yet) ...
__device__ __forceinline__ float mega_ssq_fetch(const MegaArgs &m, int t, int lane) {
    const int nch = (m.d + kSsqChunk - 1) / kSsqChunk;
    float s = 0.f;
    for (int c = lane; c < nch; c += 32) s += m.ssq[(size_t)t * nch + c];
    return s;
}
// ... and reduce them; same value in every lane
__device__ __forceinline__ float mega_inv_rms_finish(const MegaArgs &m, float s) {
    return rsqrtf(warp_sum(s) / (float)m.d + m.eps);
}
__device__ __forceinline__ float mega_inv_rms_warp(const MegaArgs &m, int t, int lane) {
    return mega_inv_rms_finish(m, mega_ssq_fetch(m, t, lane));
}

// a3: q,k,v = projection / rms; rotate q,k; append K,V to the sequence's pages.  One warp per (row, head).
__device__ void ew_qkv(const MegaArgs &m, MegaShared &sh, const MegaGemm &g, int pool_layer, int gw, int ngw, int lane) {
    const StageArgs &a = m.a;
    const int hd = m.hd, half = hd / 2, heads = m.hq + 2 * m.hkv, nq = m.hq * hd;
    const size_t stride = (size_t)m.T_pad * g.N;
    for (int item = gw; item < m.T_pad * heads; item += ngw) {
        const int t = qdiv(item, heads), h = item - t * heads, b = qdiv(t, a.R_pad), j = t - b * a.R_pad;
        if (j >= sh.nr[b]) {
            if (h < m.hq)
                for (int i = lane; i < hd; i += 32) m.q[(size_t)t * nq + h * hd + i] = 0.f;
            continue;
        }
        const float ssq = mega_ssq_fetch(m, t, lane);
        const int pos = sh.p0[b] + j;
        const int lp = qdiv(pos, a.page_size), slot = pos - lp * a.page_size;
        // only loaded here: the check of the page id (a branch with a side effect) comes after the slot loads, which
        // must not wait for this load's round trip
        const long long page = m.block_table[(size_t)b * a.max_pages + lp];
        // a head's columns lie in one 128-row weight tile (head_dim 64 or 128): one slot range for the item
        const int ns = sh.slot_n[0][(h * hd) / kWeightTileRows];
        const float *pr = m.part + (size_t)t * g.N + h * hd;
        // lane l owns columns l + 32 e of the head (e < hd / 32; hd is 64 or 128).  Every load of the item --
        // chunk sums, rotary pair, up to eight slots of each column -- is issued before the first use.
        const int ne = hd >> 5;
        const bool rot = h < m.hq + m.hkv;
        float2 cs[2] = {make_float2(1.f, 0.f), make_float2(1.f, 0.f)};
        if (rot) {
#pragma unroll
            for (int e = 0; e < 2; ++e)
                if (e < ne / 2) cs[e] = m.rope[(size_t)t * half + lane + 32 * e];
        }
        float x[4] = {0.f, 0.f, 0.f, 0.f};
        for (int s0 = 0; s0 < ns; s0 += 8) {
            float u[4][8];
#pragma unroll
            for (int e = 0; e < 4; ++e)
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const int sidx = s0 + k < ns ? s0 + k : ns - 1;   // past the last slot: re-read it, weight zero
                    u[e][k] = e < ne ? pr[sidx * stride + lane + 32 * e] : 0.f;
                }
#pragma unroll
            for (int k = 0; k < 8; ++k)
                if (s0 + k < ns) {
#pragma unroll
                    for (int e = 0; e < 4; ++e) x[e] += u[e][k];   // slot order
                }
        }
        MEGA_STAMP(78);
        const float inv = mega_inv_rms_finish(m, ssq);
        MEGA_STAMP(79);
        const bool page_ok = page >= 0 && page < m.n_pages;
        if (!page_ok && lane == 0 && h == m.hq) atomicOr(m.status, HISPEC_ST_BOUNDS);
        const size_t page_base = (((size_t)pool_layer * m.n_pages + (page_ok ? page : 0)) * m.hkv) * a.page_size * hd;
        if (rot) {
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                if (e >= ne / 2) break;
                const int i = lane + 32 * e;
                const float x0 = x[e] * inv, x1 = (ne == 4 ? x[e + 2] : x[e + 1]) * inv;
                const float c = cs[e].x, sf = cs[e].y;
                const float r0 = x0 * c - x1 * sf, r1 = x1 * c + x0 * sf;
                if (h < m.hq) {
                    m.q[(size_t)t * nq + h * hd + i] = r0;
                    m.q[(size_t)t * nq + h * hd + i + half] = r1;
                } else if (page_ok) {
                    const size_t o = page_base + ((size_t)(h - m.hq) * a.page_size + slot) * hd;
                    m.k_pages[o + i] = __float2bfloat16_rn(r0);
                    m.k_pages[o + i + half] = __float2bfloat16_rn(r1);
                }
            }
        } else if (page_ok) {
            const int vh = h - m.hq - m.hkv;
            const size_t o = page_base + ((size_t)vh * a.page_size + slot) * hd;
#pragma unroll
            for (int e = 0; e < 4; ++e)
                if (e < ne) m.v_pages[o + lane + 32 * e] = __float2bfloat16_rn(inv * x[e]);
        }
    }
}

// a6 epilogue: act_f <- hi/lo( SiLU(gate / rms) * (up / rms) )
__device__ void ew_silu(const MegaArgs &m, const MegaShared &sh, const MegaGemm &g, int gw, int ngw, int lane) {
    const int nch = (m.ffn + kEwChunk - 1) / kEwChunk;
    for (int item = gw; item < m.T_pad * nch; item += ngw) {
        const int t = qdiv(item, nch), ch = item - t * nch;
        const int c = ch * kEwChunk + lane * 8;
        const float ssq = mega_ssq_fetch(m, t, lane);
        float gt[8], up[8], v[8];
        if (c < m.ffn) {
            sum_slots8(m, sh, 2, g, t, c, gt);
            sum_slots8(m, sh, 2, g, t, m.ffn + c, up);
        }
        const float inv = mega_inv_rms_finish(m, ssq);
        if (c >= m.ffn) continue;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const float gg = gt[i] * inv;
            v[i] = (gg / (1.0f + expf(-gg))) * (up[i] * inv);
        }
        store8_hilo(m.act_f + (size_t)t * m.ffn + c, m.act_f + ((size_t)m.T_alloc + t) * m.ffn + c, v, m.plain);
    }
}

// a4 (second half): combine the key splits of every (row, q head) in split order -> act_o hi/lo.
// One warp per (row, head), a lane per HD/32 columns.  Records are HD + 4 floats apart (16-byte aligned:
// one vector load per lane and split); the (max, sum) pairs of up to 32 splits are fetched one per lane,
// and the splits are walked in order with the weights broadcast by shuffle.
constexpr int kAttnRecPad = 4;
template <int HD>
__device__ void ew_attn_merge(const MegaArgs &m, MegaShared &sh, int gw, int ngw, int lane) {
    constexpr int E = HD / 32, REC = HD + kAttnRecPad;
    const StageArgs &a = m.a;
    const int nq = m.hq * HD;
    MEGA_STAMP(30);
    for (int item = gw; item < m.T_pad * m.hq; item += ngw) {
        const int t = qdiv(item, m.hq), h = item - t * m.hq, b = qdiv(t, a.R_pad), j = t - b * a.R_pad;
        float acc[E];
#pragma unroll
        for (int e = 0; e < E; ++e) acc[e] = 0.f;
        float inv = 0.f;
        if (j < sh.nr[b]) {
            const int n_rec = m.n_splits * m.ngrp;
            const float *base = m.attn_part + ((size_t)t * m.hq + h) * n_rec * REC;
            float L = 0.f, M = -INFINITY;
            for (int s0 = 0; s0 < n_rec; s0 += 32) {
                const int cnt = min(32, n_rec - s0);
                // every load of the batch -- the lane's slice of up to 32 records and the (max, sum) pair of record
                // s0 + lane -- is issued before the first use: one L2 round trip per batch (in groups of eight the
                // loads of a group waited for the arithmetic of the one before: four round trips)
                const float *r = base + (size_t)s0 * REC + lane * E;
                float rv[32][E];
#pragma unroll
                for (int u = 0; u < 32; ++u) {
                    if (u < cnt) {
                        if constexpr (E == 4) {
                            const float4 q4 = *reinterpret_cast<const float4 *>(r + (size_t)u * REC);
                            rv[u][0] = q4.x; rv[u][1] = q4.y; rv[u][2] = q4.z; rv[u][3] = q4.w;
                        } else {
                            const float2 q2 = *reinterpret_cast<const float2 *>(r + (size_t)u * REC);
                            rv[u][0] = q2.x; rv[u][1] = q2.y;
                        }
                    } else {
#pragma unroll
                        for (int e = 0; e < E; ++e) rv[u][e] = 0.f;
                    }
                }
                float ms = -INFINITY, ls = 0.f;   // lane u holds (max, sum) of split s0 + u
                if (lane < cnt) {
                    const float2 ml = *reinterpret_cast<const float2 *>(base + (size_t)(s0 + lane) * REC + HD);
                    ms = ml.x; ls = ml.y;
                }
                if (!(ls > 0.f)) { ms = -INFINITY; ls = 0.f; }
                float Mb = ms;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) Mb = fmaxf(Mb, __shfl_xor_sync(0xffffffffu, Mb, o));
                const float Mn = fmaxf(M, Mb);
                const float corr = (M == -INFINITY) ? 0.f : exp2f(M - Mn);   // rescale what earlier batches added
                L *= corr;
#pragma unroll
                for (int e = 0; e < E; ++e) acc[e] *= corr;
                const float wl = (ms == -INFINITY) ? 0.f : exp2f(ms - Mn);
#pragma unroll
                for (int u = 0; u < 32; ++u) {
                    if (u < cnt) {   // (warp-uniform)
                        const float w = __shfl_sync(0xffffffffu, wl, u);
                        const float l = __shfl_sync(0xffffffffu, ls, u);
                        L += l * w;
#pragma unroll
                        for (int e = 0; e < E; ++e) acc[e] += w * rv[u][e];
                    }
                }
                M = Mn;
            }
            inv = L > 0.f ? 1.0f / L : 0.f;
        }
        __nv_bfloat16 *ohi = m.act_o + (size_t)t * nq + h * HD + lane * E;
        __nv_bfloat16 *olo = m.act_o + ((size_t)m.T_alloc + t) * nq + h * HD + lane * E;
#pragma unroll
        for (int e = 0; e < E; ++e) split_hi_lo(acc[e] * inv, ohi[e], olo[e], m.plain);
        MEGA_STAMP(31);
    }
    MEGA_STAMP(32);
}

// one round of a polling loop that serves several queues with non-blocking tests: bounded, and gives up once the CTA aborts
__device__ __forceinline__ bool mega_poll_idle(uint32_t &idle, bool did, volatile int *ab, uint32_t *status) {
    if (did) { idle = 0; return true; }
    if (++idle >= (1u << 28)) { *ab = 1; atomicOr(status, HISPEC_ST_TIMEOUT); return false; }
    if ((idle & 65535u) == 0u && *ab) return false;
    return true;
}

// shared-memory address of KV page stage s: a0 + (s & 1) * d1 + (s >> 1) * d2
struct AttnSmem {
    uint32_t a0, d1, d2;
    __device__ __forceinline__ uint32_t at(int s) const { return a0 + (uint32_t)(s & 1) * d1 + (uint32_t)(s >> 1) * d2; }
};

// ---- attention phase: items (split, kv head x row group, sequence) dealt round-robin to CTAs -------
template <int HD>
__device__ void mega_attention(const CUtensorMap *tmK, const CUtensorMap *tmV, const MegaArgs &m, MegaShared &sh,
                               const AttnSmem sm_attn, int pool_layer, uint32_t &pg_it, int warp, int lane) {
    constexpr int TILE = 16 * HD * 2, KS = HD / 16, NT = HD / 8;
    const StageArgs &a = m.a;
    volatile int *abort_flag = &sh.abort_flag;
    const int per_b = m.n_splits * m.hkv * m.n_mg;
    const int n_items = per_b * a.batch;
    const int QR = m.G * a.R_pad;
    for (int item = blockIdx.x; item < n_items; item += gridDim.x) {
        const int b = qdiv(item, per_b), rest = item - b * per_b;
        const int y = qdiv(rest, m.n_splits), split = rest - y * m.n_splits;
        const int kvh = qdiv(y, m.n_mg), mg = y - kvh * m.n_mg;
        const int nr = sh.nr[b], p0 = sh.p0[b];
        const int total_pages = (p0 + nr + 15) >> 4;
        int chunk = qdiv(total_pages + m.n_splits - 1, m.n_splits);
        if (chunk < 1) chunk = 1;
        const int pg0 = split * chunk, pg1 = min(pg0 + chunk, total_pages);
        const int n_pg = (nr > 0 && pg1 > pg0) ? pg1 - pg0 : 0;
        if (warp == kWarpX || warp == kWarpMma0 + 1) {
            // Two page producers -- the activation loader's warp and the second MMA warp, both idle in this phase --
            // take the pages in turn (the number of stages is even, so a stage always belongs to the same producer):
            // one issuing thread needs ~0.4 us per page, which bounded the phase on long contexts.  (A producer warp
            // whose 16 lanes each feed one stage and poll side by side measured 1 to 2 % slower than this.)
            const uint32_t pw = warp == kWarpX ? 0u : 1u;
            // first row of this KV head in page 0 of the layer's pool, and the rows from one page to the next (a TMA
            // coordinate is 32 bits wide, so the product fits)
            const int row0 = (int)(((long long)pool_layer * m.n_pages * m.hkv + kvh) * 16), page_rows = m.hkv * 16;
            MEGA_STAMP(10);
            for (int i0 = 0; i0 < n_pg; i0 += 32) {
                const int my = i0 + lane;
                int pgid = 0;
                if (my < n_pg) pgid = m.block_table[(size_t)b * a.max_pages + pg0 + my];
                if (my < n_pg && (pgid < 0 || pgid >= m.n_pages)) { atomicOr(m.status, HISPEC_ST_BOUNDS); pgid = 0; }
                const int cnt = min(32, n_pg - i0);
                for (int u = (int)((pw - (pg_it + (uint32_t)i0)) & 1u); u < cnt; u += 2) {   // this producer's pages
                    const int page = __shfl_sync(0xffffffffu, pgid, u);
                    const uint32_t it = pg_it + i0 + u;
                    const int s = it & (uint32_t)(m.attn_stages - 1);
                    const uint32_t ph = (it >> m.attn_log2) & 1u;
                    if (lane == 0 && a_wait(a_smem_u32(&sh.a_empty[s]), ph ^ 1u, abort_flag, m.status)) {
                        const uint32_t fb = a_smem_u32(&sh.a_full[s]);
                        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(fb), "r"(2 * TILE) : "memory");
                        const int row = row0 + page * page_rows;
                        const uint32_t dk = sm_attn.at(s), dv = dk + TILE;
                        // one copy per tensor: the box spans the head dimension's 64-element halves as its third dimension
                        tma_load_3d(dk, tmK, 0, row, 0, fb);
                        tma_load_3d(dv, tmV, 0, row, 0, fb);
                    }
                }
            }
            MEGA_STAMP(12);
        } else if (warp >= kWarpEpi0) {
            MEGA_STAMP(20);
            // With one or two 16-row tiles in the item the four warps form 4 or 2 groups that take the item's
            // pages in turn; each group leaves its own record, combined with the key splits by the merge.
            const int mtp = 4 / m.ngrp;
            const int cw = (warp - kWarpEpi0) % mtp, grp = (warp - kWarpEpi0) / mtp;
            const int r_lo = mg * 64 + cw * 16 + (lane >> 2), r_hi = r_lo + 8;
            const int j_lo = qdiv(r_lo, m.G), g_lo = r_lo - j_lo * m.G, j_hi = qdiv(r_hi, m.G), g_hi = r_hi - j_hi * m.G;
            const bool v_lo = cw < m.mt && r_lo < QR && j_lo < nr, v_hi = cw < m.mt && r_hi < QR && j_hi < nr;
            const int kmax_lo = v_lo ? p0 + j_lo : -1, kmax_hi = v_hi ? p0 + j_hi : -1;
            const int nq = m.hq * HD;
            const float *q_lo = m.q + ((size_t)(b * a.R_pad + j_lo) * nq + (size_t)(kvh * m.G + g_lo) * HD);
            const float *q_hi = m.q + ((size_t)(b * a.R_pad + j_hi) * nq + (size_t)(kvh * m.G + g_hi) * HD);
            uint32_t qh[KS][4], ql[KS][4];
            const int c2 = (lane & 3) * 2;
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) {
#pragma unroll
                for (int part = 0; part < 4; ++part) {
                    const bool hi_row = part & 1;
                    const float *src = hi_row ? q_hi : q_lo;
                    const bool valid = hi_row ? v_hi : v_lo;
                    const int col = ks * 16 + c2 + ((part & 2) ? 8 : 0);
                    float x0 = 0.f, x1 = 0.f;
                    if (valid) { float2 tt = *reinterpret_cast<const float2 *>(src + col); x0 = tt.x * m.scale_log2; x1 = tt.y * m.scale_log2; }
                    const float h0 = __bfloat162float(__float2bfloat16_rn(x0)), h1 = __bfloat162float(__float2bfloat16_rn(x1));
                    qh[ks][part] = pack_bf16(x0, x1);
                    ql[ks][part] = pack_bf16(x0 - h0, x1 - h1);
                }
            }
            float o[NT][4];
#pragma unroll
            for (int n = 0; n < NT; ++n) { o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f; }
            float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;
            bool ok = true;
            const bool active = cw < m.mt;   // warps without rows only keep the page ring moving
            MEGA_STAMP(21);
            // pages go to the warp groups (1, 2 or 4 of them) in turn by their running number; the number of stages is a
            // multiple of the number of groups, so a stage always belongs to the same group and only its warps touch it
            for (int i = (int)(((uint32_t)grp - pg_it) & (uint32_t)(m.ngrp - 1)); i < n_pg && ok; i += m.ngrp) {
                const uint32_t it = pg_it + i;
                const int s = it & (uint32_t)(m.attn_stages - 1);
                const uint32_t ph = (it >> m.attn_log2) & 1u;
                ok = a_wait(a_smem_u32(&sh.a_full[s]), ph, abort_flag, m.status);
                if (!ok) break;
                MEGA_STAMP(22);
                if (active) {
                    const uint32_t sk = sm_attn.at(s), sv = sk + TILE;
                    // four independent accumulator chains (2 key tiles x hi/lo query planes), added at the end
                    float sc[2][4], sl[2][4];
#pragma unroll
                    for (int n = 0; n < 2; ++n) {
                        sc[n][0] = sc[n][1] = sc[n][2] = sc[n][3] = 0.f;
                        sl[n][0] = sl[n][1] = sl[n][2] = sl[n][3] = 0.f;
                    }
                    const int mat = lane >> 3, rin = lane & 7;
#pragma unroll
                    for (int ks = 0; ks < KS; ++ks) {
                        const int key = (mat >> 1) * 8 + rin;
                        const int chunk16 = (ks & 3) * 2 + (mat & 1);
                        const uint32_t addr = sk + (ks >> 2) * 2048 + key * 128 + ((chunk16 ^ (key & 7)) << 4);
                        uint32_t kb[4];
                        ldmatrix_x4(addr, kb);
                        mma_bf16_16816(sc[0], qh[ks], kb[0], kb[1]);
                        mma_bf16_16816(sl[0], ql[ks], kb[0], kb[1]);
                        mma_bf16_16816(sc[1], qh[ks], kb[2], kb[3]);
                        mma_bf16_16816(sl[1], ql[ks], kb[2], kb[3]);
                    }
#pragma unroll
                    for (int n = 0; n < 2; ++n)
#pragma unroll
                        for (int e = 0; e < 4; ++e) sc[n][e] += sl[n][e];
                    const int key0 = (pg0 + i) * 16;
                    float mx_lo = -INFINITY, mx_hi = -INFINITY;
#pragma unroll
                    for (int n = 0; n < 2; ++n)
#pragma unroll
                        for (int e = 0; e < 2; ++e) {
                            const int key = key0 + n * 8 + c2 + e;
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
                    const float e00 = exp2f(sc[0][0] - base_lo), e01 = exp2f(sc[0][1] - base_lo);
                    const float e02 = exp2f(sc[0][2] - base_hi), e03 = exp2f(sc[0][3] - base_hi);
                    const float e10 = exp2f(sc[1][0] - base_lo), e11 = exp2f(sc[1][1] - base_lo);
                    const float e12 = exp2f(sc[1][2] - base_hi), e13 = exp2f(sc[1][3] - base_hi);
                    uint32_t pa[4] = {pack_bf16(e00, e01), pack_bf16(e02, e03), pack_bf16(e10, e11), pack_bf16(e12, e13)};
                    l_lo = l_lo * cr_lo + (e00 + e01 + e10 + e11);
                    l_hi = l_hi * cr_hi + (e02 + e03 + e12 + e13);
#pragma unroll
                    for (int n = 0; n < NT; ++n) { o[n][0] *= cr_lo; o[n][1] *= cr_lo; o[n][2] *= cr_hi; o[n][3] *= cr_hi; }
#pragma unroll
                    for (int n = 0; n < NT; n += 2) {
                        const int key = (mat & 1) * 8 + rin;
                        const int cg = n + (mat >> 1);
                        const uint32_t addr = sv + (cg >> 3) * 2048 + key * 128 + (((cg & 7) ^ (key & 7)) << 4);
                        uint32_t vb[4];
                        ldmatrix_x4_trans(addr, vb);
                        mma_bf16_16816(o[n], pa, vb[0], vb[1]);
                        mma_bf16_16816(o[n + 1], pa, vb[2], vb[3]);
                    }
                }
                __syncwarp();
                if (lane == 0)
                    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(a_smem_u32(&sh.a_empty[s])) : "memory");
            }
            MEGA_STAMP(23);
            l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1);
            l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
            l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1);
            l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);
            if (!ok) { l_lo = l_hi = 0.f; m_lo = m_hi = -INFINITY; }
            if (v_lo) {
                float *dst = m.attn_part + (((((size_t)(b * a.R_pad + j_lo) * m.hq + kvh * m.G + g_lo) * m.n_splits + split) * m.ngrp + grp) * (HD + kAttnRecPad));
#pragma unroll
                for (int n = 0; n < NT; ++n) *reinterpret_cast<float2 *>(dst + n * 8 + c2) = make_float2(o[n][0], o[n][1]);
                if ((lane & 3) == 0) { dst[HD] = m_lo; dst[HD + 1] = l_lo; }
            }
            if (v_hi) {
                float *dst = m.attn_part + (((((size_t)(b * a.R_pad + j_hi) * m.hq + kvh * m.G + g_hi) * m.n_splits + split) * m.ngrp + grp) * (HD + kAttnRecPad));
#pragma unroll
                for (int n = 0; n < NT; ++n) *reinterpret_cast<float2 *>(dst + n * 8 + c2) = make_float2(o[n][2], o[n][3]);
                if ((lane & 3) == 0) { dst[HD] = m_hi; dst[HD + 1] = l_hi; }
            }
            MEGA_STAMP(24);
        }
        pg_it += n_pg;
    }
}

// ---- projection phase roles -----------------------------------------------------------------
struct MegaRing {
    uint32_t base;         // shared address of stage 0 of this pipeline
    uint32_t stage_bytes;  // 16 KiB weight tile + activation tile
    uint32_t x_bytes;
    int stages;
};
// slot index and phase bit of a role's running position in its ring (no division in the loops)
struct RingPos {
    int s;
    uint32_t ph;
    __device__ RingPos() : s(0), ph(0) {}
    __device__ __forceinline__ void advance(int stages) {
        if (++s == stages) { s = 0; ph ^= 1u; }
    }
};

__device__ __forceinline__ void mega_fill_seglists(const MegaArgs &m, MegaShared &sh) {
    if (threadIdx.x >= 10) return;
    const int kind = threadIdx.x >> 1, p = threadIdx.x & 1;
    const MegaGemm *g = kind < 4 ? &m.gemms[m.a.l0 * 4 + kind] : m.head;
    SegIter seg(g->tiles, g->kb_total, kind == 4, blockIdx.x, p, gridDim.x);
    SegList &L = sh.segs[kind][p];
    int n = 0, tile, kb0, kb1;
    while (n < kMegaMaxSegs && seg.next(tile, kb0, kb1)) {
        L.tile[n] = tile; L.kb0[n] = (short)kb0; L.kb1[n] = (short)kb1;
        ++n;
    }
    L.n = n;
}

// position in the call's flattened sequence of weight blocks (projection, segment, k-block) of one pipeline
struct WCursor {
    const MegaArgs *m;
    const MegaShared *sh;
    int p;
    int gi, n_g;   // projection index in call order; 4 per layer, then the exit head
    int rep;       // step of a block of draft steps (the same projections again)
    int si, tile, kb, kb1;
    bool valid;
    __device__ int kind() const { return gi + 1 < n_g ? (gi & 3) : 4; }
    __device__ const MegaGemm *gemm() const {
        return gi + 1 < n_g ? &m->gemms[(m->a.l0 + (gi >> 2)) * 4 + (gi & 3)] : m->head;
    }
    __device__ WCursor(const MegaArgs *m_, const MegaShared *sh_, int p_)
        : m(m_), sh(sh_), p(p_), gi(0), n_g(4 * (m_->a.l1 - m_->a.l0) + 1), rep(0), si(-1), tile(0), kb(0), kb1(0), valid(true) {
        advance();
    }
    __device__ void advance() {
        if (++kb < kb1) return;
        for (;;) {
            const SegList &L = sh->segs[kind()][p];
            if (++si < L.n) { tile = L.tile[si]; kb = L.kb0[si]; kb1 = L.kb1[si]; return; }
            si = -1;
            if (++gi >= n_g) {
                if (++rep >= m->n_rep) { valid = false; return; }
                gi = 0;
            }
        }
    }
};

// Both polling loops below serve the two pipelines from ONE thread with non-blocking tests: two lanes of a
// warp that spin in separate loops are not scheduled fairly (one pipeline starves), and a third warp per
// scheduler partition would cap every thread at 168 registers.

// warp 0, one thread: every weight block of the call, per pipeline in consumption order, into that
// pipeline's ring -- across projection and phase boundaries.  The first block of a projection is held back
// until the previous projection's last block has LANDED: when the ring frees up at the end of a phase every
// SM issues a ring's worth of loads at once, and without the gate the tail blocks the running phase still
// waits for queue behind 24 MB of the next phase's data (measured: +1.5 to 3 us per phase).
struct WLane {
    WCursor ld;
    RingPos pos;
    int cur_gi;
    uint32_t last_bar, last_ph;
    bool gate;
    int hold;   // attention phases that must have finished before the next block may be loaded (0: none)
    __device__ WLane(const MegaArgs *m, const MegaShared *sh, int p) : ld(m, sh, p), cur_gi(0), last_bar(0), last_ph(0), gate(false), hold(0) {
        cur_gi = ld.gi;
    }
};
// tensor map of projection number gi of the call (4 per layer, then the exit head; past the end: the first again,
// which a block of draft steps comes back to) into the descriptor cache
__device__ __forceinline__ void mega_prefetch_map(const MegaArgs &m, int gi, int n_g) {
    if (gi >= n_g) gi = 0;
    const MegaGemm *g = gi + 1 < n_g ? &m.gemms[(m.a.l0 + (gi >> 2)) * 4 + (gi & 3)] : m.head;
    asm volatile("prefetch.tensormap [%0];" ::"l"(&g->tmW) : "memory");
}
// attention phases that precede the projection the cursor stands in (only where the pages take the rings whole;
// a pipeline without blocks in some projection skips it, so every projection computes its own count)
__device__ __forceinline__ int mega_w_hold(const MegaArgs &m, const WCursor &c) {
    if (m.attn_in_ring != 2 || !c.valid) return 0;
    const int layers = m.a.l1 - m.a.l0, kind = c.kind();
    return c.rep * layers + (kind == 4 ? layers : (c.gi >> 2) + (kind >= 1 ? 1 : 0));
}
__device__ __forceinline__ bool mega_w_issue(const MegaArgs &m, int p, WLane &w, const MegaRing &ring, MegaShared &sh, uint64_t policy) {
    if (!w.ld.valid) return false;
    if (w.hold) {   // the rings hold KV pages until this CTA's attention items are done
        if (*((volatile int *)&sh.attn_epoch) < w.hold) return false;
        w.hold = 0;
    }
    if (w.gate) {
        if (!mbar_test_wait(w.last_bar, w.last_ph)) return false;
        w.gate = false;
    }
    if (!mbar_test_wait(smem_u32(&sh.empty[p][w.pos.s]), w.pos.ph ^ 1u)) return false;
#ifdef HISPEC_STAMPS
    if (p == 0 && w.ld.kb == sh.segs[w.ld.kind()][0].kb0[0] && w.ld.si == 0) MEGA_STAMP(80 + w.ld.kind());
#endif
    const uint32_t fb = smem_u32(&sh.w_full[p][w.pos.s]);
    mbar_expect_tx(fb, kWTileBytes);
    tma_load_2d_stream(ring.base + w.pos.s * ring.stage_bytes, &w.ld.gemm()->tmW, w.ld.kb * kTileK, w.ld.tile * kWeightTileRows, fb,
                       policy);
    w.last_bar = fb;
    w.last_ph = w.pos.ph;
    w.ld.advance();
    w.pos.advance(ring.stages);
    if (w.ld.valid && w.ld.gi + w.ld.rep * w.ld.n_g != w.cur_gi) {
        w.cur_gi = w.ld.gi + w.ld.rep * w.ld.n_g;
        w.gate = true;
        w.hold = mega_w_hold(m, w.ld);
        // the tensor map of the projection AFTER the one that starts now: a map's first use otherwise waits for its
        // 128 bytes to come from memory, at the head of a phase
        if (p == 0) mega_prefetch_map(m, w.ld.gi + 1, w.ld.n_g);
    }
    return true;
}
__device__ __forceinline__ void mega_w_producer(const MegaArgs &m, const MegaRing *ring, MegaShared &sh) {
    volatile int *ab = &sh.abort_flag;
    WLane w0(&m, &sh, 0), w1(&m, &sh, 1);
    mega_prefetch_map(m, 0, w0.ld.n_g);
    mega_prefetch_map(m, 1, w0.ld.n_g);
    w0.hold = mega_w_hold(m, w0.ld);
    w1.hold = mega_w_hold(m, w1.ld);
    // weights are read exactly once per call: mark their lines evict-first so that they do not push the
    // partial sums, activations and KV pages (which are re-read) out of L2
    const uint64_t policy = l2_policy_evict_first();
    uint32_t idle = 0;
    while (w0.ld.valid || w1.ld.valid) {
        const bool d0 = mega_w_issue(m, 0, w0, ring[0], sh, policy);
        const bool d1 = mega_w_issue(m, 1, w1, ring[1], sh, policy);
        if (!mega_poll_idle(idle, d0 || d1, ab, m.status)) return;
    }
}

// warp 3, one thread: the activation operand of both pipelines' k-blocks of one projection phase
struct XCursor {
    const SegList *L;
    int i, kb;
    bool valid;
    __device__ XCursor(const SegList *L_) : L(L_), i(0), kb(0), valid(L_->n > 0) {
        if (valid) kb = L->kb0[0];
        skip();
    }
    __device__ void skip() {
        while (valid && kb >= L->kb1[i]) {
            if (++i >= L->n) valid = false; else kb = L->kb0[i];
        }
    }
    __device__ void advance() { ++kb; skip(); }
};
__device__ __forceinline__ bool mega_x_load(int kind, const CUtensorMap *tmX, const MegaRing *ring, MegaShared &sh,
                                            RingPos *pos, uint32_t *status) {
    volatile int *ab = &sh.abort_flag;
    XCursor c0(&sh.segs[kind][0]), c1(&sh.segs[kind][1]);
    uint64_t policy;   // the activation operand is re-read by every CTA: keep it in L2
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(policy));
    uint32_t idle = 0;
    while (c0.valid || c1.valid) {
        bool did = false;
#pragma unroll
        for (int p = 0; p < 2; ++p) {
            XCursor &c = p ? c1 : c0;
            RingPos &ps = pos[p];
            if (c.valid && mbar_test_wait(smem_u32(&sh.empty[p][ps.s]), ps.ph ^ 1u)) {
                const uint32_t fb = smem_u32(&sh.x_full[p][ps.s]);
                mbar_expect_tx(fb, ring[p].x_bytes);
                asm volatile(
                    "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3, %4}], [%5], %6;"
                    ::"r"(ring[p].base + ps.s * ring[p].stage_bytes + kWTileBytes), "l"(tmX), "r"(c.kb * kTileK), "r"(0), "r"(0),
                    "r"(fb), "l"(policy) : "memory");
                c.advance();
                ps.advance(ring[p].stages);
                did = true;
            }
        }
        if (!mega_poll_idle(idle, did, ab, status)) return false;
    }
    return true;
}

__device__ __forceinline__ bool mega_mma(const MegaArgs &m, int kind, int p, int ncols, const MegaRing &ring, MegaShared &sh,
                                         RingPos &pos, uint32_t &seg_it, uint32_t *status) {
    volatile int *ab = &sh.abort_flag;
    const uint32_t idesc = umma_idesc_bf16(ncols);
    const SegList &L = sh.segs[kind][p];
    for (int i = 0; i < L.n; ++i) {
        const int kb0 = L.kb0[i], kb1 = L.kb1[i];
        const int buf = seg_it & 1;
        const uint32_t aph = (seg_it >> 1) & 1u;
        if (!mbar_wait(smem_u32(&sh.acc_empty[p][buf]), aph ^ 1u, ab, status)) return false;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t tmem_d = sh.tmem + (p * 2 + buf) * kMegaAccCols;
        for (int kb = kb0; kb < kb1; ++kb) {
            if (!mbar_wait(smem_u32(&sh.w_full[p][pos.s]), pos.ph, ab, status)) return false;
            if (!mbar_wait(smem_u32(&sh.x_full[p][pos.s]), pos.ph, ab, status)) return false;
            if (i == 0 && kb == kb0) MEGA_STAMP(43);
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint64_t ad = umma_desc_sw128(ring.base + pos.s * ring.stage_bytes);
            const uint64_t bd = umma_desc_sw128(ring.base + pos.s * ring.stage_bytes + kWTileBytes);
#pragma unroll
            for (int k = 0; k < kTileK / 16; ++k)
                umma_bf16(tmem_d, ad + (uint64_t)(2 * k), bd + (uint64_t)(2 * k), idesc, (kb > kb0 || k) ? 1u : 0u);
            umma_commit(smem_u32(&sh.empty[p][pos.s]));
            pos.advance(ring.stages);
        }
        umma_commit(smem_u32(&sh.acc_full[p][buf]));
        ++seg_it;
    }
    return true;
}

// accumulator columns [c0, c0 + 8) of this warp's 32 TMEM lanes, hi + lo planes added
__device__ __forceinline__ void mega_acc_ld8(uint32_t taddr, int c0, int t_box, int planes, float *v) {
    tmem_ld8(taddr + (uint32_t)c0, v);
    if (planes == 2) {
        float w[8];
        tmem_ld8(taddr + (uint32_t)(t_box + c0), w);
#pragma unroll
        for (int i = 0; i < 8; ++i) v[i] += w[i];
    }
}

// warps 4..7, split-K projections: drain the accumulators of both pipelines' segments, alternating
__device__ __forceinline__ bool mega_epilogue_part(const MegaGemm *g, int kind, const MegaArgs &m, MegaShared &sh,
                                                   uint32_t *seg_it, int warp, int lane) {
    volatile int *ab = &sh.abort_flag;
    const int lg = warp & 3;
    const SegList &L0 = sh.segs[kind][0], &L1 = sh.segs[kind][1];
    const size_t stride = (size_t)m.T_pad * g->N;
    const int rounds = L0.n > L1.n ? L0.n : L1.n;
    for (int i = 0; i < rounds; ++i) {
#pragma unroll
        for (int p = 0; p < 2; ++p) {
            const SegList &L = p ? L1 : L0;
            if (i >= L.n) continue;
            const int tile = L.tile[i];
            const int buf = seg_it[p] & 1;
            const uint32_t aph = (seg_it[p] >> 1) & 1u;
            if (!mbar_wait(smem_u32(&sh.acc_full[p][buf]), aph, ab, m.status)) return false;
            MEGA_STAMP(45);
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t taddr = sh.tmem + (p * 2 + buf) * kMegaAccCols + ((uint32_t)(lg * 32) << 16);
            const int n = tile * kWeightTileRows + lg * 32 + lane;
            const int slot = 2 * blockIdx.x + p - (int)sh.slot_first[kind][tile];
            for (int c0 = 0; c0 < m.T_pad; c0 += 8) {
                float v[8];
                mega_acc_ld8(taddr, c0, m.t_box, m.planes, v);
                if (c0 == 0) MEGA_STAMP(46);
                if (n < g->N) {
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        if (c0 + j < m.T_pad) m.part[slot * stride + (size_t)(c0 + j) * g->N + n] = v[j];
                }
            }
            MEGA_STAMP(47);
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0)
                asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(&sh.acc_empty[p][buf])) : "memory");
            ++seg_it[p];
        }
    }
    return true;
}

// optional output of the exit head: logits of eight rows (columns c0..c0+7 of the accumulators) for this thread's
// vocabulary entry; 1 / rms of the rows is taken once per warp.  Kept out of line: the hot path never runs it.
struct Float8 { float a, b, c, d, e, f, g, h; };   // passed by value: in registers
__device__ __noinline__ void mega_store_logits(const MegaArgs &m, MegaShared &sh, int N, int n, int c0, Float8 s, int lane) {
    const float v[8] = {s.a, s.b, s.c, s.d, s.e, s.f, s.g, s.h};
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int t = c0 + i;
        if (t >= m.T_pad) break;
        const float inv = mega_inv_rms_warp(m, t, lane);
        const int b = qdiv(t, m.a.R_pad), j = t - b * m.a.R_pad;
        if (n < N && j < sh.nr[b]) m.logits[((size_t)b * m.a.max_rows + j) * N + n] = v[i] * inv;
    }
}

// warps 4..7, exit head: each tile's accumulator is the sum of the two pipelines' K halves; every
// column (activation row) is reduced to its top-2 over this warp's 32 vocabulary entries
__device__ __forceinline__ bool mega_epilogue_head(const MegaGemm *g, const MegaArgs &m, MegaShared &sh,
                                                   uint32_t *seg_it, int warp, int lane) {
    volatile int *ab = &sh.abort_flag;
    const int lg = warp & 3;
    const SegList &L = sh.segs[4][0];
    for (int si = 0; si < L.n; ++si) {
        const int tile = L.tile[si];
        uint32_t taddr[2];
        int bufs[2];
#pragma unroll
        for (int p = 0; p < 2; ++p) {
            bufs[p] = seg_it[p] & 1;
            const uint32_t aph = (seg_it[p] >> 1) & 1u;
            if (!mbar_wait(smem_u32(&sh.acc_full[p][bufs[p]]), aph, ab, m.status)) return false;
            taddr[p] = sh.tmem + (p * 2 + bufs[p]) * kMegaAccCols + ((uint32_t)(lg * 32) << 16);
        }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const int n = tile * kWeightTileRows + lg * 32 + lane;
        for (int c0 = 0; c0 < m.T_pad; c0 += 8) {
            float v[8], w[8];
            mega_acc_ld8(taddr[0], c0, m.t_box, m.planes, v);
            mega_acc_ld8(taddr[1], c0, m.t_box, m.planes, w);
            if (m.logits)   // parity / sampling output: off the hot path
                mega_store_logits(m, sh, g->N, n, c0, Float8{v[0] + w[0], v[1] + w[1], v[2] + w[2], v[3] + w[3], v[4] + w[4], v[5] + w[5],
                                                             v[6] + w[6], v[7] + w[7]}, lane);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                if (c0 + i >= m.T_pad) break;
                const int t = c0 + i;
                const float val = (n < g->N) ? v[i] + w[i] : -INFINITY;
                Top2 best = top2_warp(Top2{val, -INFINITY, n < g->N ? n : 0x7fffffff});
                if (lane == 0) {
                    float *o = m.top_part + ((size_t)(tile * 4 + lg) * m.T_pad + t) * 4;
                    o[0] = best.v1; o[1] = __int_as_float(best.i1); o[2] = best.v2;
                }
            }
        }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncwarp();
#pragma unroll
        for (int p = 0; p < 2; ++p) {
            if (lane == 0)
                asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(&sh.acc_empty[p][bufs[p]])) : "memory");
            ++seg_it[p];
        }
    }
    return true;
}

// warps 4..7, after the CTA's exit-head tiles: one top-2 record per row over this CTA's own tile records, so that
// the final reduction reads gridDim.x records per row instead of four per 128 vocabulary entries
__device__ void mega_head_cta_merge(const MegaArgs &m, MegaShared &sh, int warp, int lane) {
    asm volatile("bar.sync 2, 128;" ::: "memory");   // the four epilogue warps' records are written
    const SegList &L = sh.segs[4][0];
    const int n_rec = L.n * 4;
    for (int t = warp - kWarpEpi0; t < m.T_pad; t += 4) {
        Top2 best = {-INFINITY, -INFINITY, 0x7fffffff};
        for (int i = lane; i < n_rec; i += 32) {
            const int rec = L.tile[i >> 2] * 4 + (i & 3);
            const float4 o = *reinterpret_cast<const float4 *>(m.top_part + ((size_t)rec * m.T_pad + t) * 4);
            best = top2_merge(best, Top2{o.x, o.z, __float_as_int(o.y)});
        }
        best = top2_warp(best);
        if (lane == 0)
            *reinterpret_cast<float4 *>(m.cta_top + ((size_t)blockIdx.x * m.T_pad + t) * 4) =
                make_float4(best.v1, __int_as_float(best.i1), best.v2, 0.f);
    }
}

// ---- a9 (second half) + a10 for sequence b, by the worker threads of one CTA ---------------------
__device__ void mega_accept(const MegaArgs &m, MegaShared &sh, int b, int step) {
    const StageArgs &a = m.a;
    const AcceptArgs &r = m.r;
    const int nr = sh.nr[b];
    const int lane = threadIdx.x & 31, w = (threadIdx.x >> 5) - 1;
    // one warp per row: the CTAs' records (one per CTA and row, written before the last grid barrier) in CTA order
    for (int j = w; j < nr; j += kMegaWorkers / 32) {
        const int t = b * a.R_pad + j;
        Top2 best = {-INFINITY, -INFINITY, 0x7fffffff};
        for (int c = lane; c < (int)gridDim.x; c += 32) {
            const float4 o = *reinterpret_cast<const float4 *>(m.cta_top + ((size_t)c * m.T_pad + t) * 4);
            best = top2_merge(best, Top2{o.x, o.z, __float_as_int(o.y)});
        }
        best = top2_warp(best);
        const float inv = mega_inv_rms_warp(m, t, lane);
        if (lane == 0) {
            m.argmax_ws[t] = best.i1;
            if (r.argmax_ids) r.argmax_ids[(size_t)b * a.max_rows + j] = best.i1;
            if (r.top2) {
                r.top2[((size_t)b * a.max_rows + j) * 2] = best.v1 * inv;
                r.top2[((size_t)b * a.max_rows + j) * 2 + 1] = best.v2 * inv;
            }
        }
    }
    worker_bar();
    if (threadIdx.x != kMegaLeader) return;
    const int p0 = sh.p0[b];
    if (a.mode == 1 && r.defer) return;
    if (a.mode == 1) {
        const int nd = sh.nd[b];
        int acc = 0;
        while (acc < nd && acc < nr && r.draft_tokens[(size_t)b * r.token_stride + acc] == m.argmax_ws[b * a.R_pad + acc]) ++acc;
        if (r.n_accepted) r.n_accepted[b] = acc;
        if (r.next_token) r.next_token[b] = (acc < nr) ? m.argmax_ws[b * a.R_pad + acc] : -1;
        if (r.pending && nr > 0) {
            if (acc < nr) r.pending[b] = m.argmax_ws[b * a.R_pad + acc];
            else if (acc > 0) r.pending[b] = r.draft_tokens[(size_t)b * r.token_stride + acc - 1];
        }
        if (r.tentative && a.l1 == a.L_i && nr > 0) {
            int32_t *tv = r.tentative + (size_t)b * a.max_rows + sh.dst[b];
            for (int j = 0; j < acc; ++j) tv[j] = r.draft_tokens[(size_t)b * r.token_stride + j];
            if (acc < nr) tv[acc] = m.argmax_ws[b * a.R_pad + acc];
        }
        if (nr > 0) {
            const int nl = p0 + min(acc + 1, nr);
            m.len_d[b] = nl;
            if (a.l1 > a.L_d) m.len_i[b] = nl;
            if (a.l1 > a.L_i) m.len_f[b] = nl;
        }
    } else if (nr > 0) {
        const int nl = p0 + nr;
        m.len_d[b] = nl;
        if (a.l1 > a.L_d) m.len_i[b] = nl;
        if (a.l1 > a.L_i) m.len_f[b] = nl;
        if (m.block) {   // a block of draft steps: the token feeds the next step; the bonus step's token is dropped
            if (step < m.n_steps) m.block[(size_t)b * m.block_stride + step] = m.argmax_ws[b * a.R_pad + nr - 1];
        } else if (r.out_tokens) {
            bool emit = true;
            if (r.n_tokens) emit = (nl == r.n_tokens[b]);
            if (emit) r.out_tokens[(size_t)b * r.out_stride] = m.argmax_ws[b * a.R_pad + nr - 1];
        }
    }
}

// ---- the kernel --------------------------------------------------------------------------------
template <int HD>
__global__ void __launch_bounds__(kMegaThreads, 1)
hispec_stage_kernel(const __grid_constant__ CUtensorMap tmXd, const __grid_constant__ CUtensorMap tmXo,
                    const __grid_constant__ CUtensorMap tmXf, const __grid_constant__ CUtensorMap tmK,
                    const __grid_constant__ CUtensorMap tmV, const __grid_constant__ MegaArgs m) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ MegaShared sh;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const StageArgs &a = m.a;
    const int ncols = m.t_box * m.planes;

    MegaRing ring[2];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    for (int p = 0; p < 2; ++p) {
        ring[p].x_bytes = (uint32_t)ncols * 128u;
        ring[p].stage_bytes = kWTileBytes + ring[p].x_bytes;
        ring[p].stages = m.stages;
        ring[p].base = base + p * m.stages * ring[p].stage_bytes;
    }
    // KV page staging of the attention phase: its own area behind the rings, or -- with many rows, where an
    // activation tile is at least as large as a K + V page -- the activation areas of the ring stages, which are
    // idle between two projections (that shared memory then buys another ring stage)
    AttnSmem sm_attn;
    if (m.attn_in_ring == 2) {
        sm_attn.a0 = base; sm_attn.d1 = 2 * 16 * HD * 2; sm_attn.d2 = 2 * sm_attn.d1;
    } else if (m.attn_in_ring) {
        sm_attn.a0 = ring[0].base + kWTileBytes; sm_attn.d1 = ring[1].base - ring[0].base; sm_attn.d2 = ring[0].stage_bytes;
    } else {
        sm_attn.a0 = base + 2 * m.stages * ring[0].stage_bytes; sm_attn.d1 = 2 * 16 * HD * 2; sm_attn.d2 = 2 * sm_attn.d1;
    }

    if (threadIdx.x == 0) {
        sh.abort_flag = 0;
        sh.attn_epoch = 0;
        sh.trace_n = 0;
        sh.bar_k = 0;
        sh.stamp_on = 0;
        sh.stamp_n = 0;
        if (blockIdx.x == 0) *((volatile unsigned *)m.bar_next) = 0u;
        if (m.trace && blockIdx.x == 0) {
            unsigned long long t;
            asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
            m.trace[1023] = t;
        }
        for (int p = 0; p < 2; ++p) {
            for (int s = 0; s < m.stages; ++s) {
                mbar_init(smem_u32(&sh.w_full[p][s]), 1);
                mbar_init(smem_u32(&sh.x_full[p][s]), 1);
                mbar_init(smem_u32(&sh.empty[p][s]), 1);
            }
            for (int i = 0; i < 2; ++i) {
                mbar_init(smem_u32(&sh.acc_full[p][i]), 1);
                mbar_init(smem_u32(&sh.acc_empty[p][i]), 4);
            }
        }
        for (int s = 0; s < kMegaAttnStages; ++s) {
            mbar_init(smem_u32(&sh.a_full[s]), 1);
            mbar_init(smem_u32(&sh.a_empty[s]), 4 / m.ngrp);   // the warps of the group that owns the stage
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 2) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh.tmem)), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    mega_prep_rows(m, sh, 0, threadIdx.x, blockDim.x);
    mega_fill_seglists(m, sh);
    for (int i = threadIdx.x; i < 4 * kMegaSlotTiles; i += blockDim.x) {
        const int kind = i / kMegaSlotTiles, tile = i % kMegaSlotTiles;
        const MegaGemm &g = m.gemms[m.a.l0 * 4 + kind];
        if (tile < g.tiles) {
            int first, ns;
            mega_slots(tile, g.tiles, g.kb_total, gridDim.x, first, ns);
            sh.slot_n[kind][tile] = (unsigned short)ns;
            sh.slot_first[kind][tile] = (unsigned short)first;
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");

    if (warp == 0) {
        // ---- weight producer: the whole call's weight blocks of both pipelines, in consumption order
        if (lane == 0) mega_w_producer(m, ring, sh);
    } else {
        const int gw = (warp - 1) * gridDim.x + blockIdx.x, ngw = (kMegaWorkers / 32) * gridDim.x;
        uint32_t seg_it[2] = {0, 0}, pg_it = 0;   // per-thread progress counters of the role loops
        RingPos pos, xpos[2];
        const CUtensorMap *tmX[3] = {&tmXd, &tmXo, &tmXf};
        // `head` is a compile-time tag: the layer loop holds ONE copy of the projection roles for its four
        // projections (a copy per projection made a layer's code larger than the instruction cache)
        auto gemm_phase = [&](const MegaGemm *g, int kind, int xbuf, auto head) {
            MEGA_STAMP(40 + kind);
            if (warp == kWarpMma0 || warp == kWarpMma0 + 1) {
                const int p = warp - kWarpMma0;
                if (lane == 0) mega_mma(m, kind, p, ncols, ring[p], sh, pos, seg_it[p], m.status);
            } else if (warp == kWarpX) {
                if (lane == 0) mega_x_load(kind, tmX[xbuf], ring, sh, xpos, m.status);
                __syncwarp();
            } else {
                if constexpr (decltype(head)::value) {
                    mega_epilogue_head(g, m, sh, seg_it, warp, lane);
                    mega_head_cta_merge(m, sh, warp, lane);
                } else {
                    mega_epilogue_part(g, kind, m, sh, seg_it, warp, lane);
                }
            }
            MEGA_STAMP(50 + kind);
            grid_sync(m, sh, false);   // partial sums / top-2 records: read by plain loads
        };
        for (int step = 0; step < m.n_rep; ++step) {
        if (step > 0) {   // a block of draft steps: the previous step's tokens and lengths are final after this barrier
            grid_sync(m, sh, false);
            mega_prep_rows(m, sh, step, threadIdx.x - kMegaLeader, kMegaWorkers);
            worker_bar();
        }
        ew_rows_in(m, sh, m.attn_norm[a.l0], step, gw, ngw, lane);
        ew_rope_table(m, sh, gw, ngw, lane);
        grid_sync(m, sh);
        for (int l = a.l0; l < a.l1; ++l) {
            const MegaGemm *G4 = &m.gemms[l * 4];
            const int pool_layer = l - m.first_layer;
#ifdef HISPEC_STAMPS
            if (threadIdx.x == kMegaLeader) sh.stamp_on = (l == a.l0 + 3);
#endif
#pragma unroll 1
            for (int kind = 0; kind < 4; ++kind) {
                gemm_phase(&G4[kind], kind, kind == 1 ? 1 : (kind == 3 ? 2 : 0), std::false_type{});
                if (kind == 0) {
                    MEGA_STAMP(70);
                    ew_qkv(m, sh, G4[0], pool_layer, gw, ngw, lane);
                    MEGA_STAMP(71);
                    grid_sync(m, sh);
                    mega_attention<HD>(&tmK, &tmV, m, sh, sm_attn, pool_layer, pg_it, warp, lane);
                    if (m.attn_in_ring == 2) {   // every page has been consumed: the rings go back to the weight producer
                        worker_bar();
                        if (threadIdx.x == kMegaLeader) *((volatile int *)&sh.attn_epoch) = sh.attn_epoch + 1;
                    }
                    grid_sync(m, sh, false);
                    ew_attn_merge<HD>(m, sh, gw, ngw, lane);
                } else if (kind == 2) {
                    MEGA_STAMP(74);
                    ew_silu(m, sh, G4[2], gw, ngw, lane);
                    MEGA_STAMP(75);
                } else {
                    const bool last = kind == 3 && l + 1 == a.l1;
                    const float *gain = kind == 1 ? m.ffn_norm[l] : (last ? m.final_norm : m.attn_norm[l + 1]);
                    MEGA_STAMP(72);
                    ew_resid(m, sh, G4[kind], kind, gain, last ? m.exit_buf : nullptr, last ? m.hidden_out : nullptr, gw, ngw, lane);
                    MEGA_STAMP(73);
                }
                grid_sync(m, sh);
            }
        }
        gemm_phase(m.head, 4, 0, std::true_type{});
        for (int b = blockIdx.x; b < a.batch; b += gridDim.x) mega_accept(m, sh, b, step);
        }
        if (m.trace && blockIdx.x == 0 && threadIdx.x == kMegaLeader) {   // end of CTA 0's work (it finishes sequence 0)
            unsigned long long t;
            asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
            m.trace[1022] = t;
        }
    }
    __syncthreads();
    if (warp == 2) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(sh.tmem), "r"(512u) : "memory");
    }
}

}  // namespace hispec
