// Row bookkeeping, normalisation, rotary/KV-append, SwiGLU, exit-head reduction and
// prefix-acceptance kernels, plus the plain CUDA-core GEMM kept as an on-device
// cross-check of the tensor-core path.  Row t of a call is (sequence b, row j) with
// t = b * R_pad + j; rows j >= n_rows[b] are padding and carry zeros.
#pragma once

#include "common.cuh"

namespace hispec {

// ---- programmatic dependent launch --------------------------------------------------
// Every kernel lets its successor start early and waits for its predecessor's memory
// before touching anything the predecessor wrote.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

__device__ __forceinline__ float bf16_bits_to_f32(uint16_t b) { return __uint_as_float(((uint32_t)b) << 16); }

// x ~= hi + lo with hi = bf16(x), lo = bf16(x - hi): two bf16 operands carry ~16 mantissa bits.
__device__ __forceinline__ void split_hi_lo(float x, __nv_bfloat16 &hi, __nv_bfloat16 &lo, bool plain) {
    hi = __float2bfloat16_rn(x);
    lo = plain ? __float2bfloat16_rn(0.0f) : __float2bfloat16_rn(x - __bfloat162float(hi));
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Block-wide sum in a fixed order (same result on every run).  `red` holds >= 32 floats.
__device__ __forceinline__ float block_sum(float v, float *red) {
    int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
    v = warp_sum(v);
    __syncthreads();
    if (lane == 0) red[w] = v;
    __syncthreads();
    float s = 0.0f;
    for (int i = 0; i < nw; ++i) s += red[i];
    return s;
}

struct StageArgs {
    int32_t L_d, L_i, L_f, l0, l1;
    int batch, R_pad, max_rows, max_pages, page_size;
    int mode;            // 0: rows from the embedding (draft / prefill), 1: rows from a hidden buffer (verify)
    int tok_stride, tok_offset;   // embedding mode: token of row j is tokens[b*tok_stride + tok_offset + j]
    int fixed_rows;      // embedding mode without n_tokens: rows per sequence
    int k;               // verify: upper bound of the block length
    int is_target;       // verify over [L_i, L_f)
};

// ---- per-call row bookkeeping ---------------------------------------------------------
// Decides, per sequence, the position of row 0, how many rows are valid and where exit
// rows go, and checks the length counters against the call (Sec. 3.2: the buffers must be
// aligned with the layer groups).  One thread per sequence.
__global__ void prep_rows_kernel(StageArgs a, const int32_t *len_d, const int32_t *len_i, const int32_t *len_f,
                                 const int32_t *n_rows_in, const int32_t *n_draft_in, const int32_t *tokens,
                                 const int32_t *n_tokens, RowMeta rm, uint32_t *status) {
    pdl_launch_dependents();
    pdl_wait();
    int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= a.batch) return;
    int gA = len_d[b], gB = len_i[b], gC = len_f[b];
    int p0 = a.l0 < a.L_d ? gA : (a.l0 < a.L_i ? gB : gC);
    uint32_t st = 0;
    int nr, nd = 0;
    if (a.mode == 0) {
        if (n_tokens) {
            nr = n_tokens[b] - a.tok_offset;
            nr = nr < 0 ? 0 : (nr > a.R_pad ? a.R_pad : nr);
        } else {
            nr = a.fixed_rows;
            if (tokens[b * a.tok_stride + a.tok_offset] < 0) nr = 0;  // negative id: sequence sits this call out
        }
    } else if (n_rows_in) {
        nr = n_rows_in[b];
        nd = n_draft_in[b];
        if (nr < 0 || nr > a.R_pad || nd < 0 || nd > nr || nr > nd + 1 || nd > a.k) { st |= HISPEC_ST_STATE; nr = 0; nd = 0; }
    } else {  // every row the stage below has buffered
        int avail = (a.l0 == a.L_d) ? gA - gB : gB - gC;
        if (avail < 0) avail = 0;
        if (a.is_target && avail > a.k) st |= HISPEC_ST_STATE;
        nr = avail < a.R_pad ? avail : a.R_pad;
        nd = nr < a.k ? nr : a.k;
    }
    // all layer groups the range crosses must be at the same position
    if (a.l0 < a.L_d && a.l1 > a.L_d && gB != p0) st |= HISPEC_ST_STATE;
    if (a.l0 < a.L_i && a.l1 > a.L_i && gC != p0) st |= HISPEC_ST_STATE;
    if (gC > gB || gB > gA) st |= HISPEC_ST_STATE;
    // the rows consumed must have been buffered by the stage below
    if (a.mode == 1) {
        int avail = (a.l0 == a.L_d) ? gA - gB : gB - gC;
        if (avail < nr) st |= HISPEC_ST_STATE;
    }
    int dst = (a.l1 == a.L_d) ? p0 - gB : ((a.l1 == a.L_i) ? p0 - gC : 0);
    if (a.l1 != a.L_f && (dst < 0 || dst + nr > a.max_rows)) st |= HISPEC_ST_BOUNDS;
    if ((long long)p0 + nr > (long long)a.max_pages * a.page_size || p0 < 0) st |= HISPEC_ST_BOUNDS;
    if (st) {
        atomicOr(status, st);
        nr = 0;
        nd = 0;
    }
    rm.p0[b] = p0;
    rm.n_rows[b] = nr;
    rm.n_draft[b] = nd;
    rm.dst_row[b] = dst;
}

// ---- a0 + a1: fetch rows (embedding or buffered hidden state) and apply the first RMSNorm
__global__ void rows_in_norm_kernel(StageArgs a, RowMeta rm, const int32_t *tokens, const __nv_bfloat16 *tok_emb,
                                    int vocab, const float *h_src, const float *gain, float eps, int d, float *x,
                                    __nv_bfloat16 *act, int T_alloc, int plain, uint32_t *status) {
    pdl_launch_dependents();
    pdl_wait();
    __shared__ float red[32];
    int t = blockIdx.x, b = t / a.R_pad, j = t % a.R_pad;
    bool valid = j < rm.n_rows[b];
    const float *srcf = nullptr;
    const __nv_bfloat16 *srce = nullptr;
    if (valid) {
        if (a.mode == 0) {
            int tok = tokens[b * a.tok_stride + a.tok_offset + j];
            if (tok < 0 || tok >= vocab) {
                if (threadIdx.x == 0) atomicOr(status, HISPEC_ST_BOUNDS);
                valid = false;
            } else {
                srce = tok_emb + (size_t)tok * d;
            }
        } else {
            srcf = h_src + ((size_t)b * a.max_rows + j) * d;
        }
    }
    float ss = 0.0f;
    float *xr = x + (size_t)t * d;
    for (int i = threadIdx.x; i < d; i += blockDim.x) {
        float v = 0.0f;
        if (valid) v = srcf ? srcf[i] : __bfloat162float(srce[i]);
        xr[i] = v;
        ss += v * v;
    }
    ss = block_sum(ss, red);
    float inv = rsqrtf(ss / (float)d + eps);
    __nv_bfloat16 *hi = act + (size_t)t * d, *lo = act + ((size_t)T_alloc + t) * d;
    for (int i = threadIdx.x; i < d; i += blockDim.x) {
        float v = valid ? xr[i] * inv * gain[i] : 0.0f;
        split_hi_lo(v, hi[i], lo[i], plain);
    }
}

// ---- a3: sum split-K partials of the QKV projection, rotate q and k, append K,V to pages
// grid: one block per row; thread (i, g): rotary pair i of heads g, g+G, ...
__global__ void qkv_rope_store_kernel(StageArgs a, RowMeta rm, const float *part, int splits, size_t split_stride,
                                      int hq, int hkv, int hd, const double *inv_freq, float *q_out,
                                      __nv_bfloat16 *k_pages, __nv_bfloat16 *v_pages, const int32_t *block_table,
                                      long long n_pages, int pool_layer, uint32_t *status) {
    pdl_launch_dependents();
    pdl_wait();
    int t = blockIdx.x, b = t / a.R_pad, j = t % a.R_pad;
    int nq = hq * hd, N = (hq + 2 * hkv) * hd, half = hd / 2;
    float *qr = q_out + (size_t)t * nq;
    if (j >= rm.n_rows[b]) {
        for (int i = threadIdx.x; i < nq; i += blockDim.x) qr[i] = 0.0f;
        return;
    }
    int pos = rm.p0[b] + j;
    int lp = pos / a.page_size, slot = pos % a.page_size;
    long long page = block_table[(size_t)b * a.max_pages + lp];
    bool page_ok = page >= 0 && page < n_pages;
    if (!page_ok && threadIdx.x == 0) atomicOr(status, HISPEC_ST_BOUNDS);
    size_t page_base = (((size_t)pool_layer * n_pages + (page_ok ? page : 0)) * hkv) * a.page_size * hd;
    const float *pr = part + (size_t)t * N;
    int i = threadIdx.x % half, g = threadIdx.x / half, G = blockDim.x / half;
    double sn, cs;
    sincos((double)pos * inv_freq[i], &sn, &cs);
    float c = (float)cs, s = (float)sn;
    for (int h = g; h < hq + hkv; h += G) {
        float x0 = 0.0f, x1 = 0.0f;
        for (int sp = 0; sp < splits; ++sp) {
            x0 += pr[sp * split_stride + h * hd + i];
            x1 += pr[sp * split_stride + h * hd + i + half];
        }
        float r0 = x0 * c - x1 * s, r1 = x1 * c + x0 * s;
        if (h < hq) {
            qr[h * hd + i] = r0;
            qr[h * hd + i + half] = r1;
        } else if (page_ok) {
            size_t o = page_base + ((size_t)(h - hq) * a.page_size + slot) * hd;
            k_pages[o + i] = __float2bfloat16_rn(r0);
            k_pages[o + i + half] = __float2bfloat16_rn(r1);
        }
    }
    if (page_ok) {
        for (int e = threadIdx.x; e < hkv * hd; e += blockDim.x) {
            float v = 0.0f;
            for (int sp = 0; sp < splits; ++sp) v += pr[sp * split_stride + (hq + hkv) * hd + e];
            int h = e / hd, ii = e % hd;
            v_pages[page_base + ((size_t)h * a.page_size + slot) * hd + ii] = __float2bfloat16_rn(v);
        }
    }
}

// ---- a5/a7 epilogue: residual += sum of split-K partials; then RMSNorm for the next projection;
// on the last layer also buffer the exit rows (a8)
__global__ void resid_norm_kernel(StageArgs a, RowMeta rm, const float *part, int splits, size_t split_stride,
                                  const float *gain, float eps, int d, float *x, __nv_bfloat16 *act, int T_alloc,
                                  int plain, float *exit_buf, float *hidden_out) {
    pdl_launch_dependents();
    pdl_wait();
    __shared__ float red[32];
    int t = blockIdx.x, b = t / a.R_pad, j = t % a.R_pad;
    bool valid = j < rm.n_rows[b];
    float *xr = x + (size_t)t * d;
    const float *pr = part + (size_t)t * d;
    float *e1 = (valid && exit_buf) ? exit_buf + ((size_t)b * a.max_rows + rm.dst_row[b] + j) * d : nullptr;
    float *e2 = (valid && hidden_out) ? hidden_out + ((size_t)b * a.max_rows + j) * d : nullptr;
    // four columns per thread and step (d, and with it every split's offset, is a multiple of 4); the partial sums of a
    // step are loaded four splits at a time before they are added, in split order: at 144 rows a row's partials are
    // ~150 KB and a loop that waits for every load in turn spent 28 us where the traffic needs 7
    float ss = 0.0f;
    for (int i = threadIdx.x * 4; i < d; i += blockDim.x * 4) {
        float4 v = *reinterpret_cast<const float4 *>(xr + i);
        for (int sp = 0; sp < splits; sp += 4) {
            float4 u[4];
#pragma unroll
            for (int k = 0; k < 4; ++k)
                u[k] = sp + k < splits ? *reinterpret_cast<const float4 *>(pr + (sp + k) * split_stride + i) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int k = 0; k < 4; ++k)
                if (sp + k < splits) { v.x += u[k].x; v.y += u[k].y; v.z += u[k].z; v.w += u[k].w; }
        }
        if (!valid) v = make_float4(0.f, 0.f, 0.f, 0.f);
        *reinterpret_cast<float4 *>(xr + i) = v;
        if (e1) *reinterpret_cast<float4 *>(e1 + i) = v;
        if (e2) *reinterpret_cast<float4 *>(e2 + i) = v;
        ss += (v.x * v.x + v.y * v.y) + (v.z * v.z + v.w * v.w);
    }
    ss = block_sum(ss, red);
    float inv = rsqrtf(ss / (float)d + eps);
    __nv_bfloat16 *hi = act + (size_t)t * d, *lo = act + ((size_t)T_alloc + t) * d;
    for (int i = threadIdx.x; i < d; i += blockDim.x) {
        float v = valid ? xr[i] * inv * gain[i] : 0.0f;
        split_hi_lo(v, hi[i], lo[i], plain);
    }
}

// ---- a6 epilogue: SiLU(gate) * up from the split-K partials of the gate/up projection
__global__ void silu_mul_kernel(const float *part, int splits, size_t split_stride, int ffn, __nv_bfloat16 *act,
                                int T_alloc, int plain) {
    pdl_launch_dependents();
    pdl_wait();
    int t = blockIdx.y;
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= ffn) return;
    const float *pr = part + (size_t)t * 2 * ffn;
    float g = 0.0f, u = 0.0f;
    for (int sp = 0; sp < splits; ++sp) {
        g += pr[sp * split_stride + i];
        u += pr[sp * split_stride + ffn + i];
    }
    float v = (g / (1.0f + expf(-g))) * u;
    split_hi_lo(v, act[(size_t)t * ffn + i], act[((size_t)T_alloc + t) * ffn + i], plain);
}

// ---- plain CUDA-core GEMM (debug cross-check): part[s][t][n] = sum_{k in split s} W[n][k] (hi+lo)[t][k]
// one warp per output feature; rows in groups of 8
__global__ void gemm_simt_kernel(const __nv_bfloat16 *W, const __nv_bfloat16 *act, int T_alloc, int planes, int N,
                                 int K, int row0, int rows, int kb_total, int splits, float *part,
                                 size_t split_stride, int out_ld) {
    pdl_launch_dependents();
    pdl_wait();
    int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    int sp = blockIdx.y;
    if (warp >= N) return;
    int kb0 = (int)((long long)kb_total * sp / splits), kb1 = (int)((long long)kb_total * (sp + 1) / splits);
    int k0 = kb0 * kTileK, k1 = min(K, kb1 * kTileK);
    const __nv_bfloat16 *w = W + (size_t)warp * K;
    for (int r0 = 0; r0 < rows; r0 += 8) {
        float acc[8];
#pragma unroll
        for (int r = 0; r < 8; ++r) acc[r] = 0.0f;
        for (int k = k0 + lane; k < k1; k += 32) {
            float wv = __bfloat162float(w[k]);
#pragma unroll
            for (int r = 0; r < 8; ++r) {
                if (r0 + r < rows) {
                    size_t o = (size_t)(row0 + r0 + r) * K + k;
                    float xv = __bfloat162float(act[o]);
                    if (planes == 2) xv += __bfloat162float(act[(size_t)T_alloc * K + o]);
                    acc[r] += wv * xv;
                }
            }
        }
#pragma unroll
        for (int r = 0; r < 8; ++r) {
            float v = warp_sum(acc[r]);
            if (lane == 0 && r0 + r < rows) part[sp * split_stride + (size_t)(row0 + r0 + r) * out_ld + warp] = v;
        }
    }
}

// ---- top-2 of a logits row (debug path: logits materialised by the CUDA-core GEMM)
struct Top2 {
    float v1, v2;
    int i1;
};
__device__ __forceinline__ Top2 top2_merge(Top2 a, Top2 b) {
    // larger value wins, lower id on an exact tie; second = best of the rest
    bool a_first = (a.v1 > b.v1) || (a.v1 == b.v1 && a.i1 <= b.i1);
    Top2 r;
    if (a_first) { r.v1 = a.v1; r.i1 = a.i1; r.v2 = fmaxf(a.v2, b.v1); }
    else { r.v1 = b.v1; r.i1 = b.i1; r.v2 = fmaxf(b.v2, a.v1); }
    return r;
}
__device__ __forceinline__ Top2 top2_warp(Top2 v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        Top2 w;
        w.v1 = __shfl_xor_sync(0xffffffffu, v.v1, o);
        w.v2 = __shfl_xor_sync(0xffffffffu, v.v2, o);
        w.i1 = __shfl_xor_sync(0xffffffffu, v.i1, o);
        v = top2_merge(v, w);
    }
    return v;
}

// per (tile of 128 vocabulary entries, row): top-2 of the materialised logits -> top_part
__global__ void logits_tile_top2_kernel(const float *logits, int vocab, int row0, int rows, int T_pad_total,
                                        float *top_part) {
    pdl_launch_dependents();
    pdl_wait();
    int tile = blockIdx.x, t = row0 + blockIdx.y;
    int lane = threadIdx.x;  // 32 threads
    Top2 best = {-INFINITY, -INFINITY, 0x7fffffff};
    for (int n = tile * 128 + lane; n < min(vocab, tile * 128 + 128); n += 32) {
        Top2 c = {logits[(size_t)t * vocab + n], -INFINITY, n};
        best = top2_merge(best, c);
    }
    best = top2_warp(best);
    if (lane == 0) {
        float *o = top_part + ((size_t)tile * T_pad_total + t) * 4;
        o[0] = best.v1;
        o[1] = __int_as_float(best.i1);
        o[2] = best.v2;
    }
}

// ---- a9 (second half) + a10: reduce the per-tile top-2 over the vocabulary, apply
// LeadingSubstringVerify and prune the length counters.  One block per sequence.
struct AcceptArgs {
    int32_t *len_d, *len_i, *len_f;
    const int32_t *draft_tokens;  // token j of sequence b at [b * token_stride + j]; NULL for draft / prefill
    int token_stride, out_stride;
    int32_t *n_accepted, *next_token, *argmax_ids, *out_tokens, *tentative, *pending;
    float *top2;
    const int32_t *n_tokens;  // prefill: out_tokens only from the chunk that holds the last prompt token
    int defer;                // verify calls: leave acceptance, lengths, V and the pending token to a later call
};
__global__ void head_reduce_accept_kernel(StageArgs a, RowMeta rm, const float *top_part, int n_tiles,
                                          int T_pad_total, AcceptArgs r, int32_t *argmax_ws) {
    pdl_launch_dependents();
    pdl_wait();
    int b = blockIdx.x;
    int nr = rm.n_rows[b];
    int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = blockDim.x >> 5;
    // a warp per row (rows of the sequence in turn over the block's warps): 16-byte records, a lane's loads independent
    // of one another.  (One row after the other over the whole block, with two block barriers per row, took 75 us at
    // 16 x 9 rows.)
    for (int j = w; j < nr; j += nw) {
        int t = b * a.R_pad + j;
        Top2 best = {-INFINITY, -INFINITY, 0x7fffffff};
#pragma unroll 4
        for (int tile = lane; tile < n_tiles; tile += 32) {
            const float4 o = *reinterpret_cast<const float4 *>(top_part + ((size_t)tile * T_pad_total + t) * 4);
            Top2 c = {o.x, o.z, __float_as_int(o.y)};
            best = top2_merge(best, c);
        }
        best = top2_warp(best);
        if (lane == 0) {
            argmax_ws[t] = best.i1;
            if (r.argmax_ids) r.argmax_ids[(size_t)b * a.max_rows + j] = best.i1;
            if (r.top2) {
                r.top2[((size_t)b * a.max_rows + j) * 2] = best.v1;
                r.top2[((size_t)b * a.max_rows + j) * 2 + 1] = best.v2;
            }
        }
    }
    __syncthreads();
    if (threadIdx.x != 0) return;
    int p0 = rm.p0[b];
    if (a.mode == 1 && r.defer) return;
    if (a.mode == 1) {
        int nd = rm.n_draft[b], acc = 0;
        while (acc < nd && acc < nr && r.draft_tokens[(size_t)b * r.token_stride + acc] == argmax_ws[b * a.R_pad + acc])
            ++acc;
        if (r.n_accepted) r.n_accepted[b] = acc;
        if (r.next_token) r.next_token[b] = (acc < nr) ? argmax_ws[b * a.R_pad + acc] : -1;
        if (r.pending && nr > 0) {
            if (acc < nr) r.pending[b] = argmax_ws[b * a.R_pad + acc];
            else if (acc > 0) r.pending[b] = r.draft_tokens[(size_t)b * r.token_stride + acc - 1];
        }
        if (r.tentative && a.l1 == a.L_i && nr > 0) {  // V <- V || [S_1..S_a, v_{a+1}]
            int32_t *tv = r.tentative + (size_t)b * a.max_rows + rm.dst_row[b];
            for (int j = 0; j < acc; ++j) tv[j] = r.draft_tokens[(size_t)b * r.token_stride + j];
            if (acc < nr) tv[acc] = argmax_ws[b * a.R_pad + acc];
        }
        if (nr > 0) {
            int nl = p0 + min(acc + 1, nr);
            r.len_d[b] = nl;
            if (a.l1 > a.L_d) r.len_i[b] = nl;
            if (a.l1 > a.L_i) r.len_f[b] = nl;
        }
    } else {
        if (nr > 0) {
            int nl = p0 + nr;
            r.len_d[b] = nl;
            if (a.l1 > a.L_d) r.len_i[b] = nl;
            if (a.l1 > a.L_i) r.len_f[b] = nl;
            if (r.out_tokens) {
                bool emit = true;
                if (r.n_tokens) emit = (nl == r.n_tokens[b]);  // prefill: only the chunk holding the last prompt token
                if (emit) r.out_tokens[(size_t)b * r.out_stride] = argmax_ws[b * a.R_pad + nr - 1];
            }
        }
    }
}

// optional parity output: copy materialised logits rows to the caller's [batch][max_rows][vocab]
__global__ void copy_logits_kernel(StageArgs a, RowMeta rm, const float *logits_ws, int vocab, int row0, int rows,
                                   float *dst) {
    pdl_launch_dependents();
    pdl_wait();
    int t = row0 + blockIdx.y, b = t / a.R_pad, j = t % a.R_pad;
    if (j >= rm.n_rows[b]) return;
    int n = blockIdx.x * blockDim.x + threadIdx.x;
    if (n < vocab) dst[((size_t)b * a.max_rows + j) * vocab + n] = logits_ws[(size_t)t * vocab + n];
}

}  // namespace hispec
