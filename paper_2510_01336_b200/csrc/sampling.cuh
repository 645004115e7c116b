// Rejection-sampling acceptance (App. G) and inversion sampling over a vocabulary row.
//
// A vocabulary row is cut into chunks of 1024 entries.  Four small kernels, enqueued in order:
//   rs_stats_kernel    (chunks x rows x {p,q})  softmax statistics of every chunk of every candidate row;
//   rs_decide_kernel   (one CTA per sequence)   combines the chunk statistics in chunk order, runs the sequential
//                                               accept tests (two logits per row), fixes a_b and the row to draw from;
//   rs_weight_kernel   (chunks x sequences)     chunk sums of max(0, q - p) (and of q) on that row; copies the kept
//                                               verifier rows to the stage buffer;
//   rs_pick_kernel     (one CTA per sequence)   finds the chunk and the entry that hold u * total, then applies the
//                                               verify call's state transition with the sampled outcome.
// Every sum runs in a fixed order, so results do not depend on timing.  Probabilities are fp32.
#pragma once

#include "kernels.cuh"

namespace hispec {

constexpr int kVChunk = 1024;        // vocabulary entries per chunk
constexpr int kRsThreads = 256;      // threads of the chunk kernels: 4 consecutive entries per thread
constexpr int kDecFloats = 16;       // per-sequence record passed from rs_decide_kernel on

struct RsArgs {
    int stage;                 // 0: plain sampling from q (hispec_sample), 1: intermediate, 2: target
    int L_d, L_i, L_f, k, max_rows, vocab, token_stride, chunks, rows_per_seq;
    long long p_seq_stride, q_seq_stride;   // floats between two sequences' first rows
    int32_t *len_d, *len_i, *len_f;
    const int32_t *draft_tokens;
    const float *p_logits, *q_logits, *u_accept, *u_sample;
    float inv_t;
    float *stage_logits;
    int32_t *n_accepted, *next_token, *tentative, *pending;
    int32_t *out_tokens;       // stage 0
    int out_stride;
    uint32_t *status;
    float *ws_stats;           // [2][batch][rows_per_seq][chunks][2]: (max, sum exp(z - max)) per chunk
    float *ws_dec;             // [batch][kDecFloats]
    float *ws_wsum;            // [batch][chunks][2]: sum of max(0, q - p), sum of q over the chunk
};

// sum over the block in thread order: warp shuffles (fixed tree), then the warps in order
__device__ __forceinline__ float rs_block_sum(float v, float *red) {
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    __syncthreads();
    if (lane == 0) red[w] = v;
    __syncthreads();
    float r = 0.f;
    for (int i = 0; i < (int)(blockDim.x >> 5); ++i) r += red[i];
    return r;
}
__device__ __forceinline__ float rs_block_max(float v, float *red) {
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    __syncthreads();
    if (lane == 0) red[w] = v;
    __syncthreads();
    float r = red[0];
    for (int i = 1; i < (int)(blockDim.x >> 5); ++i) r = fmaxf(r, red[i]);
    return r;
}

// grid (chunks, batch * rows_per_seq, 2): z = 0 proposal rows (skipped when there are none), z = 1 verifier rows
__global__ void __launch_bounds__(kRsThreads) rs_stats_kernel(RsArgs r) {
    __shared__ float red[kRsThreads / 32];
    const int chunk = blockIdx.x, row = blockIdx.y, which = blockIdx.z;
    const float *base = which ? r.q_logits : r.p_logits;
    if (!base) return;
    const int b = row / r.rows_per_seq, j = row % r.rows_per_seq;
    const float *src = base + (size_t)b * (which ? r.q_seq_stride : r.p_seq_stride) + (size_t)j * r.vocab;
    const int v0 = chunk * kVChunk + threadIdx.x * 4;
    float z[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) z[i] = v0 + i < r.vocab ? src[v0 + i] * r.inv_t : -INFINITY;
    const float mx = rs_block_max(fmaxf(fmaxf(z[0], z[1]), fmaxf(z[2], z[3])), red);
    float s = 0.f;
    if (mx > -INFINITY) {
#pragma unroll
        for (int i = 0; i < 4; ++i) s += expf(z[i] - mx);
    }
    s = rs_block_sum(s, red);
    if (threadIdx.x == 0) {
        float *o = r.ws_stats + ((((size_t)which * gridDim.y + row) * r.chunks + chunk) * 2);
        o[0] = mx; o[1] = s;
    }
}

// (max, 1 / sum) of a whole row from its chunk records, by one warp: chunk order within a lane, then a fixed tree
__device__ __forceinline__ float2 rs_combine(const float *rec, int chunks, int lane) {
    float mx = -INFINITY;
    for (int c = lane; c < chunks; c += 32) mx = fmaxf(mx, rec[2 * c]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    float s = 0.f;
    for (int c = lane; c < chunks; c += 32)
        if (rec[2 * c] > -INFINITY) s += rec[2 * c + 1] * expf(rec[2 * c] - mx);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    return make_float2(mx, 1.0f / s);
}

// one CTA (256 threads) per sequence
__global__ void __launch_bounds__(256) rs_decide_kernel(RsArgs r, int batch) {
    __shared__ float2 s_q[64], s_p[64];
    const int b = blockIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int p0 = 0, nr = 1, nd = 0, dst = 0;
    if (r.stage != 0) {
        const int gA = r.len_d[b], gB = r.len_i[b], gC = r.len_f[b];
        // rows and drafts exactly as a verify call with "every buffered row" takes them
        p0 = r.stage == 1 ? gB : gC;
        const int avail = r.stage == 1 ? gA - gB : gB - gC;
        uint32_t bad = 0;
        if (gC > gB || gB > gA || avail < 0) bad |= HISPEC_ST_STATE;
        if (r.stage == 2 && avail > r.k) bad |= HISPEC_ST_STATE;
        nr = avail < r.k + 1 ? avail : r.k + 1;
        dst = r.stage == 1 ? p0 - gC : 0;
        if (nr > r.rows_per_seq || nr > r.max_rows || (r.stage == 1 && dst + nr > r.max_rows)) bad |= HISPEC_ST_BOUNDS;
        if (bad) {
            if (threadIdx.x == 0) atomicOr(r.status, bad);
            nr = 0;
        }
        nd = nr < r.k ? nr : r.k;
    }
    const size_t rows_total = (size_t)batch * r.rows_per_seq;
    for (int j = warp; j < nr && j < 64; j += (int)(blockDim.x >> 5)) {
        const size_t row = (size_t)b * r.rows_per_seq + j;
        const float2 q = rs_combine(r.ws_stats + ((rows_total + row) * r.chunks) * 2, r.chunks, lane);
        float2 p = q;
        if (r.p_logits && j < nd) p = rs_combine(r.ws_stats + (row * r.chunks) * 2, r.chunks, lane);
        if (lane == 0) { s_q[j] = q; s_p[j] = p; }
    }
    __syncthreads();
    if (threadIdx.x != 0) return;
    int acc = 0;
    for (; acc < nd; ++acc) {
        const int tok = r.draft_tokens[(size_t)b * r.token_stride + acc];
        if (tok < 0 || tok >= r.vocab) { atomicOr(r.status, HISPEC_ST_BOUNDS); break; }
        const float ql = r.q_logits[(size_t)b * r.q_seq_stride + (size_t)acc * r.vocab + tok];
        const float pl = r.p_logits[(size_t)b * r.p_seq_stride + (size_t)acc * r.vocab + tok];
        const float qv = expf(ql * r.inv_t - s_q[acc].x) * s_q[acc].y, pv = expf(pl * r.inv_t - s_p[acc].x) * s_p[acc].y;
        const float ratio = pv > 0.f ? fminf(1.0f, qv / pv) : 1.0f;
        if (!(r.u_accept[(size_t)b * r.max_rows + acc] < ratio)) break;
    }
    float *d = r.ws_dec + (size_t)b * kDecFloats;
    const bool draw = acc < nr;            // row `acc` was computed: replacement (acc < nd) or bonus token (acc == nd)
    const bool have_p = draw && acc < nd && r.p_logits != nullptr;
    d[0] = __int_as_float(acc); d[1] = __int_as_float(nr); d[2] = __int_as_float(nd); d[3] = __int_as_float(p0);
    d[4] = __int_as_float(dst); d[5] = __int_as_float(draw ? 1 : 0); d[6] = __int_as_float(have_p ? 1 : 0);
    if (draw) { d[7] = s_q[acc].x; d[8] = s_q[acc].y; d[9] = s_p[acc].x; d[10] = s_p[acc].y; }
}

__device__ __forceinline__ float rs_weight(const RsArgs &r, const float *qrow, const float *prow, const float *d, int v, bool use_p) {
    float w = expf(qrow[v] * r.inv_t - d[7]) * d[8];
    if (use_p) w = fmaxf(0.f, w - expf(prow[v] * r.inv_t - d[9]) * d[10]);
    return w;
}

// grid (chunks, batch)
__global__ void __launch_bounds__(kRsThreads) rs_weight_kernel(RsArgs r) {
    __shared__ float red[kRsThreads / 32];
    const int chunk = blockIdx.x, b = blockIdx.y;
    const float *d = r.ws_dec + (size_t)b * kDecFloats;
    const int acc = __float_as_int(d[0]), nr = __float_as_int(d[1]), dst = __float_as_int(d[4]);
    const bool draw = __float_as_int(d[5]) != 0, have_p = __float_as_int(d[6]) != 0;
    const int v0 = chunk * kVChunk + threadIdx.x * 4;
    if (r.stage == 1 && r.stage_logits && nr > 0) {   // proposal rows of what is kept, for the target stage
        const int rows = min(acc + 1, nr);
        for (int j = 0; j < rows; ++j) {
            const float *src = r.q_logits + (size_t)b * r.q_seq_stride + (size_t)j * r.vocab;
            float *dp = r.stage_logits + (size_t)b * r.q_seq_stride + (size_t)(dst + j) * r.vocab;
#pragma unroll
            for (int i = 0; i < 4; ++i)
                if (v0 + i < r.vocab) dp[v0 + i] = src[v0 + i];
        }
    }
    if (!draw) return;   // uniform across the block
    const float *qrow = r.q_logits + (size_t)b * r.q_seq_stride + (size_t)acc * r.vocab;
    const float *prow = have_p ? r.p_logits + (size_t)b * r.p_seq_stride + (size_t)acc * r.vocab : nullptr;
    float wr = 0.f, wq = 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i)
        if (v0 + i < r.vocab) {
            wr += rs_weight(r, qrow, prow, d, v0 + i, have_p);
            wq += rs_weight(r, qrow, prow, d, v0 + i, false);
        }
    wr = rs_block_sum(wr, red);
    wq = rs_block_sum(wq, red);
    if (threadIdx.x == 0) {
        float *o = r.ws_wsum + ((size_t)b * r.chunks + chunk) * 2;
        o[0] = wr; o[1] = wq;
    }
}

// one CTA (kRsThreads) per sequence
__global__ void __launch_bounds__(kRsThreads) rs_pick_kernel(RsArgs r) {
    __shared__ float s_w[kVChunk], s_part[32];
    __shared__ int s_chunk, s_use_p;
    __shared__ float s_lo, s_target;
    const int b = blockIdx.x;
    const float *d = r.ws_dec + (size_t)b * kDecFloats;
    const int acc = __float_as_int(d[0]), nr = __float_as_int(d[1]), p0 = __float_as_int(d[3]), dst = __float_as_int(d[4]);
    const bool draw = __float_as_int(d[5]) != 0, have_p = __float_as_int(d[6]) != 0;
    int nxt = -1;
    if (draw) {
        const float *wsg = r.ws_wsum + (size_t)b * r.chunks * 2;
        // the chunk sums go to shared memory first (parallel loads); the scan itself is sequential, in chunk order
        const bool staged = 2 * r.chunks <= kVChunk;
        if (staged)
            for (int i = threadIdx.x; i < 2 * r.chunks; i += blockDim.x) s_w[i] = wsg[i];
        __syncthreads();
        if (threadIdx.x == 0) {
            const float *ws = staged ? s_w : wsg;
            float total = 0.f;
            for (int c = 0; c < r.chunks; ++c) total += ws[2 * c];
            int use_p = have_p ? 1 : 0, col = 0;
            if (!have_p || !(total > 0.f)) {   // bonus row, or p == q left nothing over: draw from q
                use_p = 0; col = 1; total = 0.f;
                for (int c = 0; c < r.chunks; ++c) total += ws[2 * c + 1];
            }
            const float target = r.u_sample[b] * total;
            float run = 0.f;
            int pick = -1;
            for (int c = 0; c < r.chunks; ++c) {
                const float x = ws[2 * c + col];
                if (x > 0.f) {
                    pick = c;                      // last chunk of positive weight so far
                    if (target < run + x) break;
                }
                run += x;
            }
            if (pick >= 0 && pick < r.chunks) {   // the start of the chosen chunk's range
                run = 0.f;
                for (int c = 0; c < pick; ++c) run += ws[2 * c + col];
            }
            s_chunk = pick; s_use_p = use_p; s_lo = run; s_target = target;
        }
        __syncthreads();
        const int chunk = s_chunk;
        if (chunk >= 0) {
            const float *qrow = r.q_logits + (size_t)b * r.q_seq_stride + (size_t)acc * r.vocab;
            const float *prow = have_p ? r.p_logits + (size_t)b * r.p_seq_stride + (size_t)acc * r.vocab : nullptr;
            for (int i = threadIdx.x; i < kVChunk; i += blockDim.x) {
                const int v = chunk * kVChunk + i;
                s_w[i] = v < r.vocab ? rs_weight(r, qrow, prow, d, v, s_use_p != 0) : 0.f;
            }
            __syncthreads();
            // two levels inside the chunk: 32 slices of 32 entries summed by the lanes of warp 0, then one walk over
            // the slice sums and one over the chosen slice (96 sequential steps instead of 1024)
            if (threadIdx.x < 32) {
                float part = 0.f;
                for (int i = 0; i < 32; ++i) part += s_w[threadIdx.x * 32 + i];
                s_part[threadIdx.x] = part;
            }
            __syncthreads();
            if (threadIdx.x == 0) {
                float run = s_lo;
                int sl = -1;
                for (int i = 0; i < 32; ++i)
                    if (s_part[i] > 0.f) {
                        sl = i;                    // last slice of positive weight so far
                        if (s_target < run + s_part[i]) break;
                        run += s_part[i];
                    }
                int pick = -1;
                if (sl >= 0) {
                    run = s_lo;
                    for (int i = 0; i < sl; ++i) run += s_part[i];
                    for (int i = sl * 32; i < sl * 32 + 32; ++i)
                        if (s_w[i] > 0.f) {
                            pick = i;              // last entry of positive weight so far
                            run += s_w[i];
                            if (s_target < run) break;
                        }
                }
                nxt = pick >= 0 ? chunk * kVChunk + pick : 0;
            }
        } else if (threadIdx.x == 0) {
            nxt = 0;
        }
    }
    if (threadIdx.x != 0) return;
    if (r.stage == 0) {
        r.out_tokens[(size_t)b * r.out_stride] = nxt;
        return;
    }
    // the state transition of a verify call (Sec. 3.2 pruning), with the sampled outcome
    if (r.n_accepted) r.n_accepted[b] = acc;
    if (r.next_token) r.next_token[b] = nxt;
    if (r.pending && nr > 0) {
        if (acc < nr) r.pending[b] = nxt;
        else if (acc > 0) r.pending[b] = r.draft_tokens[(size_t)b * r.token_stride + acc - 1];
    }
    if (r.tentative && r.stage == 1 && nr > 0) {
        int32_t *tv = r.tentative + (size_t)b * r.max_rows + dst;
        for (int j = 0; j < acc; ++j) tv[j] = r.draft_tokens[(size_t)b * r.token_stride + j];
        if (acc < nr) tv[acc] = nxt;
    }
    if (nr > 0) {
        const int nl = p0 + min(acc + 1, nr);
        r.len_d[b] = nl;
        r.len_i[b] = nl;
        if (r.stage == 2) r.len_f[b] = nl;
    }
}

}  // namespace hispec
