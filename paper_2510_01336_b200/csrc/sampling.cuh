// Rejection-sampling acceptance (App. G) and inversion sampling over a vocabulary row.
// One CTA of 1024 threads per sequence; all reductions run in a fixed order, so results do not depend on timing.
#pragma once

#include "kernels.cuh"

namespace hispec {

constexpr int kSampleThreads = 1024;

struct RowStats {
    float mx, inv_sum;   // max of the scaled logits, 1 / sum exp(z - max)
};

__device__ __forceinline__ float block_reduce_max(float v, float *red) {
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
__device__ __forceinline__ float block_reduce_sum(float v, float *red) {
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    __syncthreads();
    if (lane == 0) red[w] = v;
    __syncthreads();
    float r = 0.f;
    for (int i = 0; i < (int)(blockDim.x >> 5); ++i) r += red[i];   // warp order
    return r;
}

// softmax statistics of one row of logits scaled by inv_t
__device__ RowStats row_stats(const float *row, int V, float inv_t, float *red) {
    float mx = -INFINITY;
    for (int v = threadIdx.x; v < V; v += blockDim.x) mx = fmaxf(mx, row[v] * inv_t);
    mx = block_reduce_max(mx, red);
    float s = 0.f;
    for (int v = threadIdx.x; v < V; v += blockDim.x) s += expf(row[v] * inv_t - mx);
    s = block_reduce_sum(s, red);
    return RowStats{mx, 1.0f / s};
}
__device__ __forceinline__ float row_prob(const float *row, int v, float inv_t, RowStats st) {
    return expf(row[v] * inv_t - st.mx) * st.inv_sum;
}

// Inversion sampling from w(v) = max(0, q(v) - p(v)) (p == nullptr: w = q), vocabulary order.  Thread t owns
// the contiguous slice [t * chunk, (t + 1) * chunk); slice sums are scanned in thread order.  Returns the
// token in every thread.  If the weights sum to zero (p == q) the draw falls back to q.
__device__ int sample_residual(const float *q_row, RowStats qs, const float *p_row, RowStats ps, int V, float inv_t, float u,
                               float *red, float *scan, int *s_tok) {
    const int chunk = (V + blockDim.x - 1) / blockDim.x;
    const int v0 = threadIdx.x * chunk, v1 = min(V, v0 + chunk);
    for (int pass = 0; pass < 2; ++pass) {
        const bool use_p = p_row != nullptr && pass == 0;
        float mine = 0.f;
        for (int v = v0; v < v1; ++v) {
            float w = row_prob(q_row, v, inv_t, qs);
            if (use_p) w = fmaxf(0.f, w - row_prob(p_row, v, inv_t, ps));
            mine += w;
        }
        __syncthreads();
        scan[threadIdx.x] = mine;
        __syncthreads();
        if (threadIdx.x == 0) {   // exclusive scan in thread order (1024 adds; the row reads above dominate)
            float run = 0.f;
            for (int i = 0; i < (int)blockDim.x; ++i) { const float x = scan[i]; scan[i] = run; run += x; }
            red[0] = run;
            *s_tok = -1;
        }
        __syncthreads();
        const float total = red[0];
        if (!(total > 0.f)) {
            if (use_p) continue;      // nothing left over: draw from q
            if (threadIdx.x == 0) *s_tok = 0;
            __syncthreads();
            return *s_tok;
        }
        const float target = u * total;
        const float lo = scan[threadIdx.x], hi = (threadIdx.x + 1 < blockDim.x) ? scan[threadIdx.x + 1] : total;
        // the slice whose cumulative range holds the target; the last non-empty slice also takes target == total
        if (mine > 0.f && target >= lo && (target < hi || (hi >= total))) {
            float run = lo;
            int pick = -1;
            for (int v = v0; v < v1; ++v) {
                float w = row_prob(q_row, v, inv_t, qs);
                if (use_p) w = fmaxf(0.f, w - row_prob(p_row, v, inv_t, ps));
                if (w > 0.f) {
                    pick = v;                       // last entry of positive weight seen so far
                    run += w;
                    if (target < run) break;
                }
            }
            if (pick >= 0) atomicMax(s_tok, pick);   // at most a few slices qualify (ties at slice borders): take one deterministically
        }
        __syncthreads();
        if (*s_tok >= 0) return *s_tok;
    }
    return 0;
}

struct SampleArgs {
    const float *logits;
    long long row_stride;
    const float *u;
    float inv_t;
    int vocab;
    int32_t *out_tokens;
    int out_stride;
};
__global__ void __launch_bounds__(kSampleThreads) sample_kernel(SampleArgs s) {
    __shared__ float red[32], scan[kSampleThreads];
    __shared__ int s_tok;
    const int b = blockIdx.x;
    const float *row = s.logits + (size_t)b * s.row_stride;
    const RowStats st = row_stats(row, s.vocab, s.inv_t, red);
    const int tok = sample_residual(row, st, nullptr, st, s.vocab, s.inv_t, s.u[b], red, scan, &s_tok);
    if (threadIdx.x == 0) s.out_tokens[(size_t)b * s.out_stride] = tok;
}

struct RejectArgs {
    int stage;                 // 1: intermediate, 2: target
    int L_d, L_i, L_f, k, max_rows, vocab, token_stride;
    int32_t *len_d, *len_i, *len_f;
    const int32_t *draft_tokens;
    const float *p_logits, *q_logits, *u_accept, *u_sample;
    float inv_t;
    float *stage_logits;
    int32_t *n_accepted, *next_token, *tentative, *pending;
    uint32_t *status;
};
__global__ void __launch_bounds__(kSampleThreads) rejection_accept_kernel(RejectArgs r) {
    __shared__ float red[32], scan[kSampleThreads];
    __shared__ int s_tok, s_acc;
    const int b = blockIdx.x;
    const int gA = r.len_d[b], gB = r.len_i[b], gC = r.len_f[b];
    // rows and drafts exactly as a verify call with "every buffered row" takes them
    const int p0 = r.stage == 1 ? gB : gC;
    int avail = r.stage == 1 ? gA - gB : gB - gC;
    uint32_t bad = 0;
    if (gC > gB || gB > gA || avail < 0) bad |= HISPEC_ST_STATE;
    if (r.stage == 2 && avail > r.k) bad |= HISPEC_ST_STATE;
    int nr = avail < r.k + 1 ? avail : r.k + 1;
    if (nr > r.max_rows) bad |= HISPEC_ST_BOUNDS;
    const int dst = r.stage == 1 ? p0 - gC : 0;
    if (r.stage == 1 && dst + nr > r.max_rows) bad |= HISPEC_ST_BOUNDS;
    if (bad) {
        if (threadIdx.x == 0) atomicOr(r.status, bad);
        nr = 0;
    }
    const int nd = nr < r.k ? nr : r.k;
    const size_t base = (size_t)b * r.max_rows * r.vocab;
    int acc = 0;
    for (; acc < nd; ++acc) {
        const int tok = r.draft_tokens[(size_t)b * r.token_stride + acc];
        const float *qrow = r.q_logits + base + (size_t)acc * r.vocab, *prow = r.p_logits + base + (size_t)acc * r.vocab;
        const RowStats qs = row_stats(qrow, r.vocab, r.inv_t, red), ps = row_stats(prow, r.vocab, r.inv_t, red);
        if (threadIdx.x == 0) {
            bool keep = false;
            if (tok >= 0 && tok < r.vocab) {
                const float qv = row_prob(qrow, tok, r.inv_t, qs), pv = row_prob(prow, tok, r.inv_t, ps);
                const float ratio = pv > 0.f ? fminf(1.0f, qv / pv) : 1.0f;
                keep = r.u_accept[(size_t)b * r.max_rows + acc] < ratio;
            } else {
                atomicOr(r.status, HISPEC_ST_BOUNDS);
            }
            s_acc = keep ? 1 : 0;
        }
        __syncthreads();
        const bool keep = s_acc != 0;
        __syncthreads();
        if (!keep) break;
    }
    int nxt = -1;
    if (acc < nr) {   // row `acc` was computed: replacement (acc < nd) or bonus token (acc == nd)
        const float *qrow = r.q_logits + base + (size_t)acc * r.vocab;
        const float *prow = acc < nd ? r.p_logits + base + (size_t)acc * r.vocab : nullptr;
        const RowStats qs = row_stats(qrow, r.vocab, r.inv_t, red);
        const RowStats ps = prow ? row_stats(prow, r.vocab, r.inv_t, red) : qs;
        nxt = sample_residual(qrow, qs, prow, ps, r.vocab, r.inv_t, r.u_sample[b], red, scan, &s_tok);
    }
    // stage 1: the proposal rows of what was kept go where the kept exit rows went (for stage 2)
    if (r.stage == 1 && r.stage_logits && nr > 0) {
        const int rows = min(acc + 1, nr);
        const float *src = r.q_logits + base;
        float *dstp = r.stage_logits + base + (size_t)dst * r.vocab;
        for (size_t i = threadIdx.x; i < (size_t)rows * r.vocab; i += blockDim.x) dstp[i] = src[i];
    }
    if (threadIdx.x != 0) return;
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
