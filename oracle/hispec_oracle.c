/*
 * CPU oracle for the HiSpec verification path -- TEST INFRASTRUCTURE ONLY.
 *
 * Plain, slow, single-precision restatement of what one partial forward pass
 * of an early-exit decoder computes (Sec. 3.1 of the paper: hidden states at an
 * exit layer L in {L_d, L_i, L_f} are projected through a shared LM head and the
 * greedy token is the argmax).  The product's CUDA path shares nothing with
 * this file; only tests, the smoke check and the bench's CPU-baseline leg may
 * load it.
 *
 * Arithmetic: fp32 throughout (the benchmark spec fixes an fp32 oracle), every
 * sum taken one row at a time in index order, keys in position order, so that a
 * row's result does not depend on which call or batch computed it.  RoPE
 * angles are formed in double precision from the integer position and then
 * rounded to fp32 (the paper is silent on this; see the readings list).
 * Weights are either fp32 or bf16 bit patterns widened exactly to fp32.
 * With kv_round_bf16 set, K (after RoPE) and V are rounded to bf16 (round to
 * nearest even) when they are stored -- the KV cache format the GPU path is
 * required to use -- and are read back as those rounded values by every row,
 * including the rows of the block being verified.
 *
 * The decoder block is the pre-norm Llama block: RMSNorm, q/k/v projections,
 * rotary embedding (rotate-half pairing), causal softmax attention with
 * grouped KV heads, output projection + residual, RMSNorm, SwiGLU FFN +
 * residual.  OpenMP only distributes independent output elements over cores.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
    int32_t n_layers, d_model, n_q_heads, n_kv_heads, head_dim, d_ffn, vocab;
    float rope_base, rms_eps;
    int32_t weights_bf16;  /* 1: matrices are uint16 bf16 patterns; 0: float */
    int32_t kv_round_bf16; /* 1: round stored K,V to bf16 */
    const void *tok_emb;   /* [vocab][d] */
    const void *const *wqkv, *const *wo, *const *wgu, *const *wdown; /* [n_layers] -> row-major [out][in] */
    const float *const *attn_norm, *const *ffn_norm;                 /* [n_layers] -> [d] */
    const float *final_norm;                                         /* [d] */
} oracle_model;

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

static inline float bf16_to_f32(uint16_t b) {
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

/* round-to-nearest-even fp32 -> bf16 -> fp32 */
float oracle_round_bf16(float x) {
    uint32_t u;
    memcpy(&u, &x, 4);
    if ((u & 0x7fffffffu) > 0x7f800000u) return x; /* NaN */
    u += 0x7fffu + ((u >> 16) & 1u);
    u &= 0xffff0000u;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

/* y = sum_k W[row][k] * x[k], k ascending */
static float dot_row(const void *W, int bf16, int64_t row, int K, const float *x) {
    float acc = 0.0f;
    if (bf16) {
        const uint16_t *w = (const uint16_t *)W + row * (int64_t)K;
        for (int k = 0; k < K; ++k) acc += bf16_to_f32(w[k]) * x[k];
    } else {
        const float *w = (const float *)W + row * (int64_t)K;
        for (int k = 0; k < K; ++k) acc += w[k] * x[k];
    }
    return acc;
}

/* out[n] = W[n][:] . x  for n in [0,N) */
static void matvec(const void *W, int bf16, int N, int K, const float *x, float *out) {
#pragma omp parallel for schedule(static)
    for (int n = 0; n < N; ++n) out[n] = dot_row(W, bf16, n, K, x);
}

/* RMSNorm: out = x / sqrt(mean(x^2) + eps) * g */
void oracle_rmsnorm(const float *x, const float *g, int d, float eps, float *out) {
    float ss = 0.0f;
    for (int i = 0; i < d; ++i) ss += x[i] * x[i];
    float inv = 1.0f / sqrtf(ss / (float)d + eps);
    for (int i = 0; i < d; ++i) out[i] = x[i] * inv * g[i];
}

/* rotary embedding of one head vector at absolute position pos:
 * pair (i, i + hd/2) is rotated by angle pos * base^(-2i/hd). */
void oracle_rope(float *v, int hd, int64_t pos, float base) {
    int half = hd / 2;
    for (int i = 0; i < half; ++i) {
        double inv_freq = pow((double)base, -2.0 * (double)i / (double)hd);
        double ang = (double)pos * inv_freq;
        float c = (float)cos(ang), s = (float)sin(ang);
        float a = v[i], b = v[i + half];
        v[i] = a * c - b * s;
        v[i + half] = b * c + a * s;
    }
}

void oracle_embed(const oracle_model *m, int32_t token, float *out) {
    int d = m->d_model;
    if (m->weights_bf16) {
        const uint16_t *e = (const uint16_t *)m->tok_emb + (int64_t)token * d;
        for (int i = 0; i < d; ++i) out[i] = bf16_to_f32(e[i]);
    } else {
        memcpy(out, (const float *)m->tok_emb + (int64_t)token * d, sizeof(float) * d);
    }
}

/*
 * One decoder layer applied to R rows of ONE sequence.
 *   x       [R][d]  residual stream, in/out
 *   p0      absolute position of row 0 (row j sits at p0 + j)
 *   kc, vc  this layer's cache, [capacity][n_kv_heads][head_dim] fp32; entries
 *           for positions < p0 must be valid; positions p0..p0+R-1 are written.
 * Row j attends to positions 0..p0+j (its own K,V included): the causal mask
 * inside the block being verified, everything cached before it.
 */
void oracle_layer(const oracle_model *m, int layer, float *x, int R, int64_t p0, float *kc, float *vc) {
    const int d = m->d_model, hq = m->n_q_heads, hkv = m->n_kv_heads, hd = m->head_dim, f = m->d_ffn;
    const int bf = m->weights_bf16;
    const int qkv_rows = (hq + 2 * hkv) * hd;
    const int group = hq / hkv;
    float *a = (float *)malloc(sizeof(float) * d);
    float *qkv = (float *)malloc(sizeof(float) * qkv_rows);
    float *q_all = (float *)malloc(sizeof(float) * (size_t)R * hq * hd);
    float *o = (float *)malloc(sizeof(float) * hq * hd);
    float *t = (float *)malloc(sizeof(float) * (d > 2 * f ? d : 2 * f));
    float *act = (float *)malloc(sizeof(float) * f);

    /* projections + RoPE + cache append, row by row */
    for (int j = 0; j < R; ++j) {
        int64_t pos = p0 + j;
        oracle_rmsnorm(x + (size_t)j * d, m->attn_norm[layer], d, m->rms_eps, a);
        matvec(m->wqkv[layer], bf, qkv_rows, d, a, qkv);
        for (int h = 0; h < hq; ++h) oracle_rope(qkv + h * hd, hd, pos, m->rope_base);
        for (int h = 0; h < hkv; ++h) oracle_rope(qkv + (hq + h) * hd, hd, pos, m->rope_base);
        memcpy(q_all + (size_t)j * hq * hd, qkv, sizeof(float) * hq * hd);
        float *kdst = kc + (size_t)pos * hkv * hd, *vdst = vc + (size_t)pos * hkv * hd;
        const float *ksrc = qkv + hq * hd, *vsrc = qkv + (hq + hkv) * hd;
        for (int i = 0; i < hkv * hd; ++i) {
            kdst[i] = m->kv_round_bf16 ? oracle_round_bf16(ksrc[i]) : ksrc[i];
            vdst[i] = m->kv_round_bf16 ? oracle_round_bf16(vsrc[i]) : vsrc[i];
        }
    }

    const float scale = 1.0f / sqrtf((float)hd);
    for (int j = 0; j < R; ++j) {
        int64_t n_keys = p0 + j + 1;
        const float *q = q_all + (size_t)j * hq * hd;
        /* softmax(q k^T / sqrt(hd)) v, per query head, keys in position order */
#pragma omp parallel for schedule(static)
        for (int h = 0; h < hq; ++h) {
            int kvh = h / group;
            float *s = (float *)malloc(sizeof(float) * (size_t)n_keys);
            float mx = -INFINITY;
            for (int64_t p = 0; p < n_keys; ++p) {
                const float *kp = kc + ((size_t)p * hkv + kvh) * hd;
                float acc = 0.0f;
                for (int i = 0; i < hd; ++i) acc += q[h * hd + i] * kp[i];
                s[p] = acc * scale;
                if (s[p] > mx) mx = s[p];
            }
            float den = 0.0f;
            for (int64_t p = 0; p < n_keys; ++p) {
                s[p] = expf(s[p] - mx);
                den += s[p];
            }
            for (int i = 0; i < hd; ++i) {
                float acc = 0.0f;
                for (int64_t p = 0; p < n_keys; ++p) acc += s[p] * vc[((size_t)p * hkv + kvh) * hd + i];
                o[h * hd + i] = acc / den;
            }
            free(s);
        }
        float *xr = x + (size_t)j * d;
        matvec(m->wo[layer], bf, d, hq * hd, o, t);
        for (int i = 0; i < d; ++i) xr[i] += t[i];

        /* SwiGLU FFN: down( silu(gate(a)) * up(a) ) */
        oracle_rmsnorm(xr, m->ffn_norm[layer], d, m->rms_eps, a);
        matvec(m->wgu[layer], bf, 2 * f, d, a, t);
        for (int i = 0; i < f; ++i) {
            float g = t[i];
            act[i] = (g / (1.0f + expf(-g))) * t[f + i];
        }
        matvec(m->wdown[layer], bf, d, f, act, t);
        for (int i = 0; i < d; ++i) xr[i] += t[i];
    }
    free(a); free(qkv); free(q_all); free(o); free(t); free(act);
}

/*
 * Layers [l0, l1) on R rows of one sequence.  kcache/vcache hold all layers:
 * [n_layers][capacity][n_kv_heads][head_dim]; only layers l0..l1-1 are touched.
 */
void oracle_forward(const oracle_model *m, int l0, int l1, float *x, int R, int64_t p0,
                    float *kcache, float *vcache, int64_t capacity) {
    size_t lstride = (size_t)capacity * m->n_kv_heads * m->head_dim;
    for (int l = l0; l < l1; ++l) oracle_layer(m, l, x, R, p0, kcache + lstride * l, vcache + lstride * l);
}

/* Exit head: logits = Whead . RMSNorm(h; final_norm)   (shared norm + head at every exit) */
void oracle_exit_logits(const oracle_model *m, const void *head, const float *h, float *logits) {
    float *a = (float *)malloc(sizeof(float) * m->d_model);
    oracle_rmsnorm(h, m->final_norm, m->d_model, m->rms_eps, a);
    matvec(head, m->weights_bf16, m->vocab, m->d_model, a, logits);
    free(a);
}

/* greedy token: largest logit, lowest id on an exact tie; also the runner-up value */
int32_t oracle_argmax(const float *logits, int n, float *top1, float *top2) {
    int32_t best = 0;
    float b1 = logits[0], b2 = -INFINITY;
    for (int i = 1; i < n; ++i) {
        if (logits[i] > b1) { b2 = b1; b1 = logits[i]; best = i; }
        else if (logits[i] > b2) b2 = logits[i];
    }
    if (top1) *top1 = b1;
    if (top2) *top2 = b2;
    return best;
}
