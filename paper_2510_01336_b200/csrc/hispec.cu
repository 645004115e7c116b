// C ABI of the HiSpec verification library: context, argument checks and the launch
// sequence of one stage call (steps a0..a10: row fetch, per layer [RMSNorm, QKV, RoPE + KV
// append, paged causal attention, O + residual, RMSNorm, SwiGLU, down + residual], exit rows,
// exit head + argmax, prefix acceptance + prune).
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <cmath>
#include <new>
#include <vector>

#include "attention.cuh"
#include "common.cuh"
#include "gemm_tc.cuh"
#include "kernels.cuh"
#include "mega.cuh"
#include "sampling.cuh"

using namespace hispec;

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            return nullptr;
        fn = (EncodeTiledFn)p;
    }
    return fn;
}

// bf16 matrix [rows][K] row-major, box = 64 (k) x box_rows, 128-byte swizzle, OOB reads give 0
bool encode_2d(CUtensorMap *tm, const void *base, uint64_t K, uint64_t rows, uint32_t box_rows) {
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {K, rows};
    cuuint64_t strides[1] = {K * 2};
    cuuint32_t box[2] = {(cuuint32_t)kTileK, box_rows};
    cuuint32_t es[2] = {1, 1};
    return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, es,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// KV pages for the persistent kernel: [rows][halves][64] with the halves as the outermost box dimension
bool encode_pages3(CUtensorMap *tm, const void *base, uint64_t hd, uint64_t rows) {
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return false;
    cuuint64_t dims[3] = {(cuuint64_t)kTileK, rows, hd / kTileK};
    cuuint64_t strides[2] = {hd * 2, (cuuint64_t)kTileK * 2};
    cuuint32_t box[3] = {(cuuint32_t)kTileK, 16, (cuuint32_t)(hd / kTileK)};
    cuuint32_t es[3] = {1, 1, 1};
    return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims, strides, box, es,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// activation buffer [2 planes][T_alloc][K]
bool encode_act(CUtensorMap *tm, const void *base, uint64_t K, uint64_t T_alloc, uint32_t t_box, uint32_t planes) {
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return false;
    cuuint64_t dims[3] = {K, T_alloc, 2};
    cuuint64_t strides[2] = {K * 2, T_alloc * K * 2};
    cuuint32_t box[3] = {(cuuint32_t)kTileK, t_box, planes};
    cuuint32_t es[3] = {1, 1, 1};
    return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims, strides, box, es,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int env_int(const char *name, int dflt) {
    const char *s = getenv(name);
    return (s && *s) ? atoi(s) : dflt;
}

inline int ceil_div(int a, int b) { return (a + b - 1) / b; }
inline int round_up(int a, int b) { return ceil_div(a, b) * b; }

// Key splits of the stand-alone attention kernel: about four CTAs per SM over (batch, KV head, row group).  (Filling the CTA slots
// exactly once instead -- fewer, longer CTAs -- is 2 % faster with equal contexts and 6 % slower with the ragged
// contexts of a serving batch, whose longest sequences then form the tail.)
inline int attn_splits(int sm_count, int batch, int hkv, int G, int R_pad) {
    int n_mg = ceil_div(G * R_pad, kAttnGroupRows);
    int s = ceil_div(4 * sm_count, batch * hkv * n_mg);
    if (s < 1) s = 1;
    if (s > 64) s = 64;
    return s;
}

struct ActMapCache {
    const void *base;
    int t_box, planes;
    CUtensorMap map;
};

}  // namespace

struct ProfEvent {
    cudaEvent_t a, b;
    int kind;
    double bytes;
};

struct hispec_ctx_ext {
    // persistent-kernel path
    bool mega_ok;              // cooperative launch available and the kernel fits
    MegaGemm *d_gemms;         // device [n_layers * 4 + 4]: per-layer projections, then cached exit heads
    const void *mega_heads[4];
    int n_mega_heads;
    const float **d_attn_norm, **d_ffn_norm;  // device arrays of device pointers
    float *ssq;                // [T_alloc][ceil(d / 128)] chunk sums of squares
    float *cta_top;            // [sm_count][T_alloc][4] per-CTA top-2 records of the persistent kernel
    float *rs_stats, *rs_dec, *rs_wsum;   // workspace of the sampling kernels (chunk statistics, decisions, chunk weights)
    float2 *rope;              // [T_alloc][head_dim / 2] (cos, sin) of this call's rows, filled by the persistent kernel
    unsigned *bar;             // grid barrier counters, used alternately by successive launches
    int bar_sel;
    unsigned long long *trace; // debug: phase time stamps of the persistent kernel (HISPEC_TRACE=1)
    size_t mega_part_floats[4];  // partial-sum floats per padded row the stream-K partition needs, per projection
    bool profiling;
    std::vector<ProfEvent> *prof;       // recorded since the last read
    std::vector<ProfEvent> *prof_free;  // event pairs ready for reuse
    // tmK / tmV: the page pools as rows of head_dim elements with the head dimension seen as [head_dim / 64][64];
    // box 64 x 16 x (head_dim / 64): a whole K (or V) page of one KV head in one TMA copy
    struct PageMaps { const void *k, *v; long long n_pages; int pool_layers; CUtensorMap tmK, tmV; } page_maps[4];
    int n_page_maps;
    ActMapCache act_cache[3][8];
    int act_cache_n[3];
    int T_alloc;
    int gemm_smem_budget;
    bool pdl;
};

static hispec_ctx_ext *ext_of(hispec_ctx *c);

struct hispec_ctx_full : hispec_ctx {
    hispec_ctx_ext ext;
};
static hispec_ctx_ext *ext_of(hispec_ctx *c) { return &static_cast<hispec_ctx_full *>(c)->ext; }

template <typename... KArgs, typename... Args>
static cudaError_t launch(hispec_ctx *c, cudaStream_t st, void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem,
                          Args &&...args) {
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = ext_of(c)->pdl ? 1 : 0;
    c->launches++;
    return cudaLaunchKernelEx(&cfg, kern, KArgs(args)...);
}

// event pair around one launch while profiling is on
struct ProfScope {
    hispec_ctx *c;
    cudaStream_t st;
    ProfEvent ev;
    bool on;
    ProfScope(hispec_ctx *c_, cudaStream_t st_, int kind, double bytes) : c(c_), st(st_), on(ext_of(c_)->profiling) {
        if (!on) return;
        hispec_ctx_ext *x = ext_of(c);
        if (!x->prof_free->empty()) {
            ev = x->prof_free->back();
            x->prof_free->pop_back();
        } else if (cudaEventCreate(&ev.a) != cudaSuccess || cudaEventCreate(&ev.b) != cudaSuccess) {
            on = false;
            return;
        }
        ev.kind = kind;
        ev.bytes = bytes;
        cudaEventRecord(ev.a, st);
    }
    ~ProfScope() {
        if (!on) return;
        cudaEventRecord(ev.b, st);
        ext_of(c)->prof->push_back(ev);
    }
};

static char g_last_error[640] = "";
static void note_error(const char *what, int line, cudaError_t e) {
    snprintf(g_last_error, sizeof(g_last_error), "%s (line %d): %s", what, line, cudaGetErrorString(e));
}
extern "C" const char *hispec_last_error(void) { return g_last_error; }

#define CK(expr)                              \
    do {                                      \
        cudaError_t e_ = (expr);              \
        if (e_ != cudaSuccess) {              \
            note_error(#expr, __LINE__, e_);  \
            return HISPEC_ECUDA;              \
        }                                     \
    } while (0)

extern "C" const char *hispec_strerror(int code) {
    switch (code) {
        case HISPEC_OK: return "ok";
        case HISPEC_EINVAL: return "invalid argument";
        case HISPEC_ECAPACITY: return "request exceeds the context's capacity";
        case HISPEC_ECUDA: return "CUDA call failed";
        case HISPEC_ENOMEM: return "workspace allocation failed";
        default: return "unknown error";
    }
}

extern "C" int hispec_create(const hispec_model_desc *desc, const hispec_weights *w, hispec_ctx **out) {
    if (!desc || !w || !out) return HISPEC_EINVAL;
    const hispec_model_desc &d = *desc;
    if (d.n_layers <= 0 || d.d_model <= 0 || d.n_q_heads <= 0 || d.n_kv_heads <= 0 || d.d_ffn <= 0 || d.vocab <= 0 ||
        d.page_size <= 0 || d.max_batch <= 0 || d.max_rows_per_seq <= 0 || d.max_pages_per_seq <= 0)
        return HISPEC_EINVAL;
    if (d.n_q_heads % d.n_kv_heads) return HISPEC_EINVAL;
    if (d.head_dim != 64 && d.head_dim != 128) return HISPEC_EINVAL;
    if (d.d_model % 8 || d.d_ffn % 8) return HISPEC_EINVAL;  // TMA: 16-byte row pitch
    if (d.max_rows_per_seq > kAttnMaxRows) return HISPEC_ECAPACITY;
    if (!w->tok_emb || !w->wqkv || !w->wo || !w->wgu || !w->wdown || !w->attn_norm || !w->ffn_norm || !w->final_norm)
        return HISPEC_EINVAL;

    hispec_ctx_full *c = new (std::nothrow) hispec_ctx_full();
    if (!c) return HISPEC_ENOMEM;
    memset(static_cast<hispec_ctx *>(c), 0, sizeof(hispec_ctx));
    memset(&c->ext, 0, sizeof(c->ext));
    c->ext.prof = new std::vector<ProfEvent>();
    c->ext.prof_free = new std::vector<ProfEvent>();
    c->d = d;
    if (cudaGetDevice(&c->device) != cudaSuccess) { delete c; return HISPEC_ECUDA; }
    cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, c->device);
    if (c->sm_count <= 0) c->sm_count = 148;
    const int L = d.n_layers;
    c->tok_emb = w->tok_emb;
    c->final_norm = w->final_norm;
    c->wqkv = new const void *[L]; c->wo = new const void *[L]; c->wgu = new const void *[L]; c->wdown = new const void *[L];
    c->attn_norm = new const float *[L]; c->ffn_norm = new const float *[L];
    c->tm_wqkv = new CUtensorMap[L]; c->tm_wo = new CUtensorMap[L]; c->tm_wgu = new CUtensorMap[L]; c->tm_wdown = new CUtensorMap[L];
    const int nq = d.n_q_heads * d.head_dim, nqkv = (d.n_q_heads + 2 * d.n_kv_heads) * d.head_dim;
    bool simt = (d.flags & HISPEC_FLAG_SIMT_GEMM) != 0;
    bool ok = true;
    for (int l = 0; l < L; ++l) {
        c->wqkv[l] = w->wqkv[l]; c->wo[l] = w->wo[l]; c->wgu[l] = w->wgu[l]; c->wdown[l] = w->wdown[l];
        c->attn_norm[l] = w->attn_norm[l]; c->ffn_norm[l] = w->ffn_norm[l];
        if (!simt && c->wqkv[l]) {
            ok = ok && encode_2d(&c->tm_wqkv[l], c->wqkv[l], d.d_model, nqkv, kWeightTileRows);
            ok = ok && encode_2d(&c->tm_wo[l], c->wo[l], nq, d.d_model, kWeightTileRows);
            ok = ok && encode_2d(&c->tm_wgu[l], c->wgu[l], d.d_model, 2 * (uint64_t)d.d_ffn, kWeightTileRows);
            ok = ok && encode_2d(&c->tm_wdown[l], c->wdown[l], d.d_ffn, d.d_model, kWeightTileRows);
        }
    }
    if (!ok) {
        snprintf(g_last_error, sizeof(g_last_error), "cuTensorMapEncodeTiled failed for a weight matrix");
        hispec_destroy(c);
        return HISPEC_ECUDA;
    }

    // split-K plan: enough CTAs to put every SM to work on each projection
    const int target = env_int("HISPEC_SPLIT_TARGET", c->sm_count);
    auto plan = [&](GemmKind k, int N, int K, bool allow_split) {
        GemmPlan &p = c->plan[k];
        p.N = N; p.K = K; p.tiles = ceil_div(N, kWeightTileRows); p.kb_total = ceil_div(K, kTileK);
        int s = allow_split ? target / p.tiles : 1;
        if (s < 1) s = 1;
        if (s > kMaxSplits) s = kMaxSplits;
        if (s > p.kb_total) s = p.kb_total;
        p.splits = s;
    };
    plan(G_QKV, nqkv, d.d_model, true);
    plan(G_O, d.d_model, nq, true);
    plan(G_GU, 2 * d.d_ffn, d.d_model, true);
    plan(G_DOWN, d.d_model, d.d_ffn, true);
    plan(G_HEAD, d.vocab, d.d_model, false);

    c->T_max = d.max_batch * d.max_rows_per_seq;
    const int T_alloc = round_up(c->T_max, 16);
    c->ext.T_alloc = T_alloc;
    c->ext.gemm_smem_budget = env_int("HISPEC_GEMM_SMEM", 100 * 1024);
    c->ext.pdl = !(d.flags & HISPEC_FLAG_NO_PDL);
    size_t part_floats = 0;
    for (int k = 0; k < G_HEAD; ++k) {
        size_t f = (size_t)c->plan[k].splits * T_alloc * c->plan[k].N;
        if (f > part_floats) part_floats = f;
    }
    // persistent-kernel path: stream-K partial slots per tile (one per CTA whose span touches the tile)
    {
        const int G = c->sm_count;
        for (int k = 0; k < G_HEAD; ++k) {
            const GemmPlan &p = c->plan[k];
            const long long U = (long long)p.tiles * p.kb_total;
            int smax = 1;
            (void)U;
            for (int tile = 0; tile < p.tiles; ++tile) {
                int first, ns;
                mega_slots(tile, p.tiles, p.kb_total, G, first, ns);
                if (ns > smax) smax = ns;
            }
            c->ext.mega_part_floats[k] = (size_t)smax * p.N;
            size_t f = (size_t)smax * T_alloc * p.N;
            if (f > part_floats) part_floats = f;
        }
    }
    c->part_floats = part_floats;
    // split records of the tiled attention kernel: enough for the largest (batch, splits) product
    {
        size_t worst = 0;
        for (int b = 1; b <= d.max_batch; ++b)
            for (int r = 1; r <= d.max_rows_per_seq; ++r) {
                size_t v = (size_t)attn_splits(c->sm_count, b, d.n_kv_heads, d.n_q_heads / d.n_kv_heads, r) * b * r;
                if (v > worst) worst = v;
            }
        c->attn_max_splits = (int)(worst / ((size_t)d.max_batch * d.max_rows_per_seq)) + 1;
        // the persistent kernel keeps up to 32 records per (row, head): key splits x warp groups
        if (worst < (size_t)32 * d.max_batch * d.max_rows_per_seq) worst = (size_t)32 * d.max_batch * d.max_rows_per_seq;
        c->attn_part_floats = worst * d.n_q_heads * (d.head_dim + 4);   // records padded to 16 bytes by the persistent kernel
    }
    auto alloc = [&](void **p, size_t bytes) { return cudaMalloc(p, bytes ? bytes : 16) == cudaSuccess; };
    ok = true;
    ok = ok && alloc((void **)&c->x, sizeof(float) * T_alloc * d.d_model);
    ok = ok && alloc((void **)&c->act_d, 2 * sizeof(__nv_bfloat16) * (size_t)T_alloc * d.d_model);
    ok = ok && alloc((void **)&c->act_o, 2 * sizeof(__nv_bfloat16) * (size_t)T_alloc * nq);
    ok = ok && alloc((void **)&c->act_f, 2 * sizeof(__nv_bfloat16) * (size_t)T_alloc * d.d_ffn);
    ok = ok && alloc((void **)&c->q, sizeof(float) * (size_t)T_alloc * nq);
    ok = ok && alloc((void **)&c->part, sizeof(float) * part_floats);
    ok = ok && alloc((void **)&c->attn_part, sizeof(float) * c->attn_part_floats);
    ok = ok && alloc((void **)&c->top_part, sizeof(float) * 4 * (size_t)c->plan[G_HEAD].tiles * 4 * T_alloc);
    if (simt) ok = ok && alloc((void **)&c->logits_ws, sizeof(float) * (size_t)T_alloc * d.vocab);
    ok = ok && alloc((void **)&c->inv_freq, sizeof(double) * (d.head_dim / 2));
    ok = ok && alloc((void **)&c->rows.p0, sizeof(int32_t) * d.max_batch);
    ok = ok && alloc((void **)&c->rows.n_rows, sizeof(int32_t) * d.max_batch);
    ok = ok && alloc((void **)&c->rows.n_draft, sizeof(int32_t) * d.max_batch);
    ok = ok && alloc((void **)&c->rows.dst_row, sizeof(int32_t) * d.max_batch);
    ok = ok && alloc((void **)&c->argmax_ws, sizeof(int32_t) * T_alloc);
    ok = ok && alloc((void **)&c->status, sizeof(uint32_t));
    ok = ok && alloc((void **)&c->ext.d_gemms, sizeof(MegaGemm) * (L * 4 + 4));
    ok = ok && alloc((void **)&c->ext.d_attn_norm, sizeof(float *) * L);
    ok = ok && alloc((void **)&c->ext.d_ffn_norm, sizeof(float *) * L);
    ok = ok && alloc((void **)&c->ext.ssq, sizeof(float) * (size_t)T_alloc * ceil_div(d.d_model, kSsqChunk));
    ok = ok && alloc((void **)&c->ext.rope, sizeof(float2) * (size_t)T_alloc * (d.head_dim / 2));
    ok = ok && alloc((void **)&c->ext.cta_top, sizeof(float) * 4 * (size_t)c->sm_count * T_alloc);
    {
        const size_t chunks = ceil_div(d.vocab, kVChunk);
        ok = ok && alloc((void **)&c->ext.rs_stats, sizeof(float) * 2 * 2 * chunks * (size_t)d.max_batch * d.max_rows_per_seq);
        ok = ok && alloc((void **)&c->ext.rs_dec, sizeof(float) * kDecFloats * (size_t)d.max_batch);
        ok = ok && alloc((void **)&c->ext.rs_wsum, sizeof(float) * 2 * chunks * (size_t)d.max_batch);
    }
    ok = ok && alloc((void **)&c->ext.bar, 2 * sizeof(unsigned));
    if (env_int("HISPEC_TRACE", 0)) ok = ok && alloc((void **)&c->ext.trace, 1024 * sizeof(unsigned long long));
    if (!ok) { hispec_destroy(c); return HISPEC_ENOMEM; }
    bool e = true;
    auto ck = [&](cudaError_t err, const char *what, int line) {
        if (err != cudaSuccess && e) note_error(what, line, err);
        e = e && err == cudaSuccess;
    };
#define CKB(expr) ck((expr), #expr, __LINE__)
    CKB(cudaMemset(c->status, 0, sizeof(uint32_t)));
    CKB(cudaMemset(c->act_d, 0, 2 * sizeof(__nv_bfloat16) * (size_t)T_alloc * d.d_model));
    CKB(cudaMemset(c->act_o, 0, 2 * sizeof(__nv_bfloat16) * (size_t)T_alloc * nq));
    CKB(cudaMemset(c->act_f, 0, 2 * sizeof(__nv_bfloat16) * (size_t)T_alloc * d.d_ffn));
    // rotary frequencies base^(-2i/hd) in double precision
    int half = d.head_dim / 2;
    double *f = new double[half];
    for (int i = 0; i < half; ++i) f[i] = pow((double)d.rope_base, -2.0 * (double)i / (double)d.head_dim);
    CKB(cudaMemcpy(c->inv_freq, f, sizeof(double) * half, cudaMemcpyHostToDevice));
    delete[] f;
    CKB(cudaFuncSetAttribute(gemm_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kGemmMaxDynSmem));
    CKB(cudaFuncSetAttribute(gemm_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kGemmMaxDynSmem));
    CKB(cudaMemset(c->ext.bar, 0, 2 * sizeof(unsigned)));
    CKB(cudaMemcpy(c->ext.d_attn_norm, c->attn_norm, sizeof(float *) * L, cudaMemcpyHostToDevice));
    CKB(cudaMemcpy(c->ext.d_ffn_norm, c->ffn_norm, sizeof(float *) * L, cudaMemcpyHostToDevice));
    if (!simt) {
        // device table of projection descriptors for the persistent kernel
        std::vector<MegaGemm> hg((size_t)L * 4 + 4);
        memset(hg.data(), 0, sizeof(MegaGemm) * hg.size());
        for (int l = 0; l < L; ++l) {
            const CUtensorMap *tms[4] = {&c->tm_wqkv[l], &c->tm_wo[l], &c->tm_wgu[l], &c->tm_wdown[l]};
            for (int k = 0; k < 4; ++k) {
                MegaGemm &g = hg[(size_t)l * 4 + k];
                if (c->wqkv[l]) g.tmW = *tms[k];
                g.N = c->plan[k].N; g.K = c->plan[k].K; g.tiles = c->plan[k].tiles; g.kb_total = c->plan[k].kb_total;
            }
        }
        CKB(cudaMemcpy(c->ext.d_gemms, hg.data(), sizeof(MegaGemm) * hg.size(), cudaMemcpyHostToDevice));
        CKB(cudaFuncSetAttribute(hispec_stage_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMegaMaxDynSmem));
        CKB(cudaFuncSetAttribute(hispec_stage_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMegaMaxDynSmem));
        int coop = 0;
        cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, c->device);
        c->ext.mega_ok = coop != 0 && d.page_size == 16 && d.max_batch <= kMegaMaxBatch &&
                         !(d.flags & (HISPEC_FLAG_MULTI_KERNEL | HISPEC_FLAG_ROWWARP_ATTN));
    }
#undef CKB
    if (!e) { hispec_destroy(c); return HISPEC_ECUDA; }
    *out = c;
    return HISPEC_OK;
}

extern "C" int hispec_destroy(hispec_ctx *c0) {
    if (!c0) return HISPEC_EINVAL;
    hispec_ctx_full *c = static_cast<hispec_ctx_full *>(c0);
    void *bufs[] = {c->x, c->act_d, c->act_o, c->act_f, c->q, c->part, c->attn_part, c->top_part, c->logits_ws, c->inv_freq,
                    c->rows.p0, c->rows.n_rows, c->rows.n_draft, c->rows.dst_row, c->argmax_ws, c->status,
                    c->ext.d_gemms, c->ext.d_attn_norm, c->ext.d_ffn_norm, c->ext.ssq, c->ext.bar, c->ext.trace, c->ext.rope, c->ext.cta_top, c->ext.rs_stats, c->ext.rs_dec, c->ext.rs_wsum};
    for (void *p : bufs)
        if (p) cudaFree(p);
    delete[] c->wqkv; delete[] c->wo; delete[] c->wgu; delete[] c->wdown; delete[] c->attn_norm; delete[] c->ffn_norm;
    delete[] c->tm_wqkv; delete[] c->tm_wo; delete[] c->tm_wgu; delete[] c->tm_wdown;
    for (std::vector<ProfEvent> *v : {c->ext.prof, c->ext.prof_free})
        if (v) {
            for (ProfEvent &e : *v) { cudaEventDestroy(e.a); cudaEventDestroy(e.b); }
            delete v;
        }
    delete c;
    return HISPEC_OK;
}

extern "C" int hispec_profile_enable(hispec_ctx *c, int on) {
    if (!c) return HISPEC_EINVAL;
    ext_of(c)->profiling = on != 0;
    return HISPEC_OK;
}

extern "C" int hispec_profile_read(hispec_ctx *c, void *stream, int kind, double *ms, double *bytes, int64_t *launches) {
    if (!c || !ms || !bytes || !launches) return HISPEC_EINVAL;
    CK(cudaStreamSynchronize((cudaStream_t)stream));
    hispec_ctx_ext *x = ext_of(c);
    double t = 0.0, by = 0.0;
    int64_t n = 0;
    std::vector<ProfEvent> keep;
    for (ProfEvent &e : *x->prof) {
        bool match = (kind == 0) ? (e.kind >= 10 && e.kind < 20) : (e.kind == kind);
        if (!match) { keep.push_back(e); continue; }
        float f = 0.0f;
        if (cudaEventElapsedTime(&f, e.a, e.b) == cudaSuccess) { t += f; by += e.bytes; ++n; }
        x->prof_free->push_back(e);
    }
    x->prof->swap(keep);
    *ms = t; *bytes = by; *launches = n;
    return HISPEC_OK;
}

// debug: copy the persistent kernel's phase time stamps (ns) of the last call; returns their number
extern "C" int hispec_debug_trace(hispec_ctx *c, unsigned long long *out, int cap) {
    hispec_ctx_ext *x = ext_of(c);
    if (!x->trace || cap < 1024) return 0;
    if (cudaDeviceSynchronize() != cudaSuccess) return 0;
    if (cudaMemcpy(out, x->trace, 1024 * sizeof(unsigned long long), cudaMemcpyDeviceToHost) != cudaSuccess) return 0;
    return 1024;
}

extern "C" int64_t hispec_launch_count(const hispec_ctx *c) { return c ? c->launches : 0; }

// the four sampling kernels, in order, as plain launches (each must see the previous one's results and, first of
// all, those of the deferred verify call)
static int run_sampling(hispec_ctx *c, cudaStream_t st, RsArgs &r, int batch) {
    hispec_ctx_ext *x = ext_of(c);
    r.chunks = ceil_div(r.vocab, kVChunk);
    r.ws_stats = x->rs_stats; r.ws_dec = x->rs_dec; r.ws_wsum = x->rs_wsum;
    r.status = c->status;
    rs_stats_kernel<<<dim3(r.chunks, batch * r.rows_per_seq, 2), kRsThreads, 0, st>>>(r);
    rs_decide_kernel<<<batch, 256, 0, st>>>(r, batch);
    rs_weight_kernel<<<dim3(r.chunks, batch), kRsThreads, 0, st>>>(r);
    rs_pick_kernel<<<batch, kRsThreads, 0, st>>>(r);
    c->launches += 4;
    CK(cudaGetLastError());
    return HISPEC_OK;
}

extern "C" int hispec_accept_rejection(hispec_ctx *c, void *stream, int stage, const hispec_exits *ex, const hispec_kv *kv,
                                       int batch, const int32_t *draft_tokens, int token_stride, int k, const float *p_logits,
                                       const float *q_logits, const float *u_accept, const float *u_sample,
                                       float temperature, float *stage_logits, const hispec_result *res) {
    if (!c || !ex || !kv || !draft_tokens || !p_logits || !q_logits || !u_accept || !u_sample) return HISPEC_EINVAL;
    if ((stage != 1 && stage != 2) || batch < 1 || batch > c->d.max_batch || k < 1 || k + 1 > c->d.max_rows_per_seq)
        return HISPEC_EINVAL;
    if (!(0 < ex->L_d && ex->L_d < ex->L_i && ex->L_i < ex->L_f && ex->L_f <= c->d.n_layers)) return HISPEC_EINVAL;
    if (!(temperature > 0.f) || token_stride < 1 || !kv->len_draft || !kv->len_inter || !kv->len_target) return HISPEC_EINVAL;
    RsArgs r;
    memset(&r, 0, sizeof(r));
    r.stage = stage; r.L_d = ex->L_d; r.L_i = ex->L_i; r.L_f = ex->L_f; r.k = k;
    r.max_rows = c->d.max_rows_per_seq; r.vocab = c->d.vocab; r.token_stride = token_stride;
    r.rows_per_seq = k + 1;
    r.p_seq_stride = r.q_seq_stride = (long long)c->d.max_rows_per_seq * c->d.vocab;
    r.len_d = kv->len_draft; r.len_i = kv->len_inter; r.len_f = kv->len_target;
    r.draft_tokens = draft_tokens; r.p_logits = p_logits; r.q_logits = q_logits;
    r.u_accept = u_accept; r.u_sample = u_sample; r.inv_t = 1.0f / temperature; r.stage_logits = stage_logits;
    if (res) { r.n_accepted = res->n_accepted; r.next_token = res->next_token; r.tentative = res->tentative; r.pending = res->pending; }
    return run_sampling(c, (cudaStream_t)stream, r, batch);
}

extern "C" int hispec_sample(hispec_ctx *c, void *stream, int batch, const float *logits, int64_t row_stride, const float *u,
                             float temperature, int32_t *out_tokens, int out_stride) {
    if (!c || !logits || !u || !out_tokens || batch < 1 || batch > c->d.max_batch || row_stride < c->d.vocab ||
        !(temperature > 0.f) || out_stride < 1)
        return HISPEC_EINVAL;
    RsArgs r;
    memset(&r, 0, sizeof(r));
    r.stage = 0; r.k = 0; r.max_rows = c->d.max_rows_per_seq; r.vocab = c->d.vocab; r.rows_per_seq = 1;
    r.q_seq_stride = row_stride; r.q_logits = logits; r.u_sample = u; r.inv_t = 1.0f / temperature;
    r.out_tokens = out_tokens; r.out_stride = out_stride;
    return run_sampling(c, (cudaStream_t)stream, r, batch);
}

extern "C" int hispec_device_status(hispec_ctx *c, void *stream, uint32_t *host_out) {
    if (!c || !host_out) return HISPEC_EINVAL;
    cudaStream_t st = (cudaStream_t)stream;
    CK(cudaStreamSynchronize(st));
    CK(cudaMemcpyAsync(host_out, c->status, sizeof(uint32_t), cudaMemcpyDeviceToHost, st));
    CK(cudaMemsetAsync(c->status, 0, sizeof(uint32_t), st));
    CK(cudaStreamSynchronize(st));
    if (*host_out & HISPEC_ST_TIMEOUT) {  // a kernel that gave up may have left the grid barrier half way
        CK(cudaMemset(ext_of(c)->bar, 0, 2 * sizeof(unsigned)));
        ext_of(c)->bar_sel = 0;
    }
    return HISPEC_OK;
}

// ---------------------------------------------------------------------------------------------
namespace {

const CUtensorMap *act_map(hispec_ctx *c, int which, const void *base, int K, int t_box, int planes) {
    hispec_ctx_ext *x = ext_of(c);
    for (int i = 0; i < x->act_cache_n[which]; ++i) {
        ActMapCache &m = x->act_cache[which][i];
        if (m.base == base && m.t_box == t_box && m.planes == planes) return &m.map;
    }
    int slot = x->act_cache_n[which] < 8 ? x->act_cache_n[which]++ : 7;
    ActMapCache &m = x->act_cache[which][slot];
    if (!encode_act(&m.map, base, K, x->T_alloc, t_box, planes)) return nullptr;
    m.base = base; m.t_box = t_box; m.planes = planes;
    return &m.map;
}

// TMA descriptors over the caller's K and V page pools: rows = (layer, page, kv head, slot), box = one
// page of one KV head, 64 dims wide
const hispec_ctx_ext::PageMaps *page_maps(hispec_ctx *c, const hispec_kv &kv) {
    hispec_ctx_ext *x = ext_of(c);
    for (int i = 0; i < x->n_page_maps; ++i) {
        auto &m = x->page_maps[i];
        if (m.k == kv.k_pages && m.v == kv.v_pages && m.n_pages == kv.n_pages && m.pool_layers == kv.n_pool_layers)
            return &m;
    }
    int slot = x->n_page_maps < 4 ? x->n_page_maps++ : 3;
    auto &m = x->page_maps[slot];
    uint64_t rows = (uint64_t)kv.n_pool_layers * kv.n_pages * c->d.n_kv_heads * c->d.page_size;
    // (the kernels address a page row through a 32-bit TMA coordinate)
    if (rows > 0x7fffffffull || !encode_pages3(&m.tmK, kv.k_pages, c->d.head_dim, rows) ||
        !encode_pages3(&m.tmV, kv.v_pages, c->d.head_dim, rows)) {
        x->n_page_maps = slot;
        return nullptr;
    }
    m.k = kv.k_pages; m.v = kv.v_pages; m.n_pages = kv.n_pages; m.pool_layers = kv.n_pool_layers;
    return &m;
}

const CUtensorMap *head_map(hispec_ctx *c, const void *head) {
    for (int i = 0; i < c->n_head_maps; ++i)
        if (c->head_maps[i].ptr == head) return &c->head_maps[i].map;
    int slot = c->n_head_maps < 4 ? c->n_head_maps++ : 3;
    if (!encode_2d(&c->head_maps[slot].map, head, c->d.d_model, c->d.vocab, kWeightTileRows)) return nullptr;
    c->head_maps[slot].ptr = head;
    return &c->head_maps[slot].map;
}

struct StageCall {
    StageArgs a;
    const hispec_exits *exits;
    const hispec_kv *kv;
    const hispec_hidden *hidden;
    const int32_t *tokens;     // embedding mode
    const int32_t *n_tokens;   // prefill
    const int32_t *draft_tokens, *n_draft, *n_rows;
    int token_stride, out_stride;
    const hispec_result *res;
    int32_t *out_tokens;
    // a block of draft steps in one launch (0 steps: a plain call)
    int32_t *block;
    int block_stride, n_steps, bonus;
};

// one projection: activation buffer `which` (0: act_d, 1: act_o, 2: act_f) times weight matrix
// *splits_used (may be NULL) receives the number of split-K partial slots written per output element
int run_gemm(hispec_ctx *c, cudaStream_t st, GemmKind kind, const void *W, const CUtensorMap *tmW, int which,
             int T_pad, const StageCall &sc, int *splits_used = nullptr) {
    const GemmPlan &p = c->plan[kind];
    hispec_ctx_ext *x = ext_of(c);
    const bool plain = (c->d.flags & HISPEC_FLAG_PLAIN_ACT) != 0;
    const bool simt = (c->d.flags & HISPEC_FLAG_SIMT_GEMM) != 0;
    const int planes = plain ? 1 : 2;
    const __nv_bfloat16 *act = which == 0 ? c->act_d : (which == 1 ? c->act_o : c->act_f);
    const bool head = kind == G_HEAD;
    const size_t split_stride = (size_t)T_pad * p.N;
    if (!head && (size_t)p.splits * split_stride > c->part_floats) return HISPEC_ECAPACITY;
    // Between 129 and 160 rows with hi/lo planes (a serving batch of 16 with k = 8): two weight tiles per CTA share
    // an activation tile (gemm_pair_kernel), one CTA per SM; the K range is split so that the grid still fills the
    // GPU once.  Up to 128 rows the one-tile kernel (one MMA over both planes, two CTAs per SM) measured 2 % faster;
    // above 160 rows three stages of the pair no longer fit and it measured 4 % slower.
    // rows one launch can take: 256 (with hi/lo planes beyond 128 rows: one MMA per plane); more rows are cut into equal
    // chunks (288 rows: 2 x 144, each in the pair kernel's window, instead of 256 + 32 -- every chunk streams the weights)
    const int n_chunks = ceil_div(T_pad, 256);
    const int chunk = T_pad <= 256 ? 256 : round_up(ceil_div(T_pad, n_chunks), 16);
    const int pair_rows = T_pad < chunk ? T_pad : chunk;
    const bool pair_mode = !simt && planes == 2 && T_pad > 128 &&
                           3 * (2 * kWTileBytes + round_up(pair_rows, 16) * planes * 128) + 1024 <= kGemmMaxDynSmem;
    int splits = head ? 1 : p.splits;
    if (pair_mode && !head) {
        const int pairs = ceil_div(p.tiles, 2);
        splits = (c->sm_count + pairs / 2) / pairs;
        if (splits < 1) splits = 1;
        if (splits > kMaxSplits) splits = kMaxSplits;
        if (splits > p.kb_total / 4) splits = p.kb_total / 4 > 0 ? p.kb_total / 4 : 1;
        while (splits > 1 && (size_t)splits * split_stride > c->part_floats) --splits;
    }
    if (splits_used) *splits_used = splits;
    for (int row0 = 0; row0 < T_pad; row0 += chunk) {
        int rows = T_pad - row0 < chunk ? T_pad - row0 : chunk;
        ProfScope prof(c, st, 10 + (int)kind, 2.0 * (double)p.N * (double)p.K);
        if (simt) {
            float *outp = head ? c->logits_ws : c->part;
            dim3 grid(ceil_div(p.N * 32, 256), head ? 1 : p.splits);
            CK(launch(c, st, gemm_simt_kernel, grid, dim3(256), 0, (const __nv_bfloat16 *)W, act, x->T_alloc, planes, p.N,
                      p.K, row0, rows, p.kb_total, head ? 1 : p.splits, outp, split_stride, p.N));
            if (head) {
                CK(launch(c, st, logits_tile_top2_kernel, dim3(p.tiles, rows), dim3(32), 0, (const float *)c->logits_ws,
                          p.N, row0, rows, T_pad, c->top_part));
                if (sc.res && sc.res->logits)
                    CK(launch(c, st, copy_logits_kernel, dim3(ceil_div(p.N, 256), rows), dim3(256), 0, sc.a, c->rows,
                              (const float *)c->logits_ws, p.N, row0, rows, sc.res->logits));
            }
            continue;
        }
        GemmArgs g;
        memset(&g, 0, sizeof(g));
        g.N = p.N; g.K = p.K; g.kb_total = p.kb_total; g.splits = splits;
        g.row0 = row0; g.rows = rows;
        g.planes = planes;
        if (pair_mode) {
            g.t_box = round_up(rows, 16);
            const int stage_bytes = 2 * kWTileBytes + g.t_box * planes * 128;
            int stages = (kGemmMaxDynSmem - 1024) / stage_bytes;
            if (stages < 2) return HISPEC_ECAPACITY;
            if (stages > 16) stages = 16;
            g.stages = stages;
            g.tmem_cols = 512;
            g.head = head ? 1 : 0;
            g.part = c->part; g.split_stride = split_stride;
            g.top_part = c->top_part; g.T_pad = T_pad;
            g.logits = (head && sc.res) ? sc.res->logits : nullptr;
            g.R_pad = sc.a.R_pad; g.max_rows = sc.a.max_rows; g.n_rows = c->rows.n_rows;
            g.status = c->status;
            const CUtensorMap *tmXp = act_map(c, which, act, p.K, g.t_box, planes);
            if (!tmXp || !tmW) return HISPEC_ECUDA;
            CK(launch(c, st, gemm_pair_kernel, dim3(ceil_div(p.tiles, 2), splits), dim3(kGemmThreads),
                      (size_t)stages * stage_bytes + 1024, *tmW, *tmXp, g));
            continue;
        }
        g.split_planes = (planes == 2 && rows > 128) ? 1 : 0;
        g.t_box = round_up(rows, (planes == 2 && !g.split_planes) ? 8 : 16);
        int ncols = g.t_box * planes;
        int tc = 32;
        while (tc < ncols) tc <<= 1;
        if (g.split_planes) tc = 512;
        g.tmem_cols = tc;
        int stage_bytes = kWTileBytes + ncols * 128;
        int stages = x->gemm_smem_budget / stage_bytes;
        if (stages < 2) stages = 2;
        if (stages > 16) stages = 16;
        while (stages > 2 && (size_t)stages * stage_bytes + 1024 > (size_t)kGemmMaxDynSmem) --stages;
        g.stages = stages;
        g.head = head ? 1 : 0;
        g.part = c->part; g.split_stride = split_stride;
        g.top_part = c->top_part; g.T_pad = T_pad;
        g.logits = (head && sc.res) ? sc.res->logits : nullptr;
        g.R_pad = sc.a.R_pad; g.max_rows = sc.a.max_rows; g.n_rows = c->rows.n_rows;
        g.status = c->status;
        const CUtensorMap *tmX = act_map(c, which, act, p.K, g.t_box, planes);
        if (!tmX || !tmW) return HISPEC_ECUDA;
        size_t smem = (size_t)stages * stage_bytes + 1024;
        CK(launch(c, st, gemm_tc_kernel, dim3(p.tiles, g.splits), dim3(kGemmThreads), smem, *tmW, *tmX, g));
    }
    return HISPEC_OK;
}

// index of the exit head's descriptor in the device table (encoded and uploaded on first use)
int mega_head_slot(hispec_ctx *c, const void *head) {
    hispec_ctx_ext *x = ext_of(c);
    for (int i = 0; i < x->n_mega_heads; ++i)
        if (x->mega_heads[i] == head) return i;
    int slot = x->n_mega_heads < 4 ? x->n_mega_heads : 3;
    MegaGemm g;
    memset(&g, 0, sizeof(g));
    if (!encode_2d(&g.tmW, head, c->d.d_model, c->d.vocab, kWeightTileRows)) return -1;
    const GemmPlan &p = c->plan[G_HEAD];
    g.N = p.N; g.K = p.K; g.tiles = p.tiles; g.kb_total = p.kb_total;
    if (cudaMemcpy(x->d_gemms + (size_t)c->d.n_layers * 4 + slot, &g, sizeof(g), cudaMemcpyHostToDevice) != cudaSuccess)
        return -1;
    x->mega_heads[slot] = head;
    if (x->n_mega_heads < 4) x->n_mega_heads++;
    return slot;
}

// the whole call as one cooperative launch of the persistent kernel; returns 1 if the call does not fit it
int run_stage_mega(hispec_ctx *c, cudaStream_t st, const StageCall &sc) {
    const hispec_model_desc &d = c->d;
    hispec_ctx_ext *x = ext_of(c);
    const StageArgs &a = sc.a;
    const int T_pad = a.batch * a.R_pad;
    const int plain = (d.flags & HISPEC_FLAG_PLAIN_ACT) ? 1 : 0;
    const int planes = plain ? 1 : 2;
    if (!x->mega_ok || T_pad * planes > kMegaAccCols) return 1;
    const hispec_kv &kv = *sc.kv;
    // The persistent kernel is built for calls dominated by the weight stream.  When the KV cache
    // a layer may have to read (by the block-table capacity; the lengths live on the device) outweighs
    // the layer's weights, the stand-alone attention kernel with its deeper page pipeline serves better.
    const double kv_cap = (double)a.batch * d.max_pages_per_seq * d.page_size * 4.0 * d.n_kv_heads * d.head_dim;
    double w_layer = 0.0;
    for (int k = 0; k < G_HEAD; ++k) w_layer += 2.0 * (double)c->plan[k].N * c->plan[k].K;
    if (kv_cap > w_layer && !env_int("HISPEC_FORCE_MEGA", 0)) return 1;
    // the kernel's index arithmetic takes quotients of positions and item numbers below 2^21 through the reciprocal unit
    if ((long long)d.max_pages_per_seq * d.page_size >= (1ll << 21)) return 1;
    MegaArgs m;
    memset(&m, 0, sizeof(m));
    m.a = a;
    m.gemms = x->d_gemms;
    const void *head = (a.l1 == a.L_d) ? sc.exits->head_d : ((a.l1 == a.L_i) ? sc.exits->head_i : sc.exits->head_f);
    int hs = mega_head_slot(c, head);
    if (hs < 0) return HISPEC_ECUDA;
    m.head = x->d_gemms + (size_t)d.n_layers * 4 + hs;
    m.attn_norm = x->d_attn_norm; m.ffn_norm = x->d_ffn_norm; m.final_norm = c->final_norm;
    m.d = d.d_model; m.hq = d.n_q_heads; m.hkv = d.n_kv_heads; m.hd = d.head_dim; m.ffn = d.d_ffn; m.vocab = d.vocab;
    m.eps = d.rms_eps;
    m.T_pad = T_pad; m.T_alloc = x->T_alloc; m.planes = planes; m.plain = plain;
    m.t_box = round_up(T_pad, planes == 2 ? 8 : 16);
    const int ncols = m.t_box * planes;
    const int stage_bytes = kWTileBytes + ncols * 128;
    // Four ring stages per pipeline: three cost 2 % (less of the next projection prefetched while the grid waits),
    // five and more cost 1 % (the longer burst of prefetch loads at the end of a projection delays the latency-bound
    // element-wise phase beside it; Llama-3-8B shape, kernel time +-0.1 %).
    // KV page staging of the attention phase (a K + V page of one KV head is 8 KB at head_dim 128):
    //  - weight-dominated calls: four pages in flight, in the ring's idle activation areas where those are large
    //    enough (32 rows and more), else in an area of their own; the weight producer prefetches the output
    //    projection into the rings meanwhile;
    //  - calls whose KV cache per layer may reach a tenth of the layer's weights: the attention phase is bound by the
    //    bytes it has in flight, so it takes both rings whole (up to kMegaAttnStages pages) and the weight producer
    //    waits for it; the output projection's first blocks then arrive during the split merge.
    const int page_bytes = 2 * 16 * d.head_dim * 2;
    const int budget = kMegaMaxDynSmem - 1024;
    const int cap = env_int("HISPEC_MEGA_STAGES", 4);
    const bool kv_heavy = kv_cap >= 0.1 * w_layer && !env_int("HISPEC_NO_WIDE", 0);
    m.attn_in_ring = kv_heavy ? 2 : ((ncols * 128 >= page_bytes) ? 1 : 0);
    int stages = (budget - (m.attn_in_ring ? 0 : 4 * page_bytes)) / (2 * stage_bytes);
    if (stages > cap) stages = cap;
    if (stages > kMegaMaxStages) stages = kMegaMaxStages;
    if (stages < 2) return 1;
    m.attn_stages = m.attn_in_ring == 2 ? 2 * stages * stage_bytes / page_bytes : 4;
    if (m.attn_stages > kMegaAttnStages) m.attn_stages = kMegaAttnStages;
    // a power of two: the two page producers and the warp groups (1, 2 or 4) divide it, and the kernel shifts and masks
    m.attn_log2 = 2;
    while ((2 << m.attn_log2) <= m.attn_stages) ++m.attn_log2;
    m.attn_stages = 1 << m.attn_log2;
    const int attn_bytes = m.attn_in_ring ? 0 : 4 * page_bytes;
    m.stages = stages;
    for (int k = 0; k < G_HEAD; ++k) {
        if (x->mega_part_floats[k] * (size_t)T_pad > c->part_floats) return 1;
        if (c->plan[k].tiles > kMegaSlotTiles) return 1;   // the kernel tabulates the partial-slot range of every tile
        // the kernel's partition arithmetic is 32-bit and its per-pipeline segment lists are fixed-size
        if ((long long)c->plan[k].tiles * c->plan[k].kb_total * 2 * c->sm_count >= (1ll << 31)) return 1;
        if (ceil_div(ceil_div(c->plan[k].tiles * c->plan[k].kb_total, 2 * c->sm_count), c->plan[k].kb_total) + 2 > kMegaMaxSegs) return 1;
    }
    if (ceil_div(c->plan[G_HEAD].tiles, c->sm_count) > kMegaMaxSegs) return 1;
    m.len_d = kv.len_draft; m.len_i = kv.len_inter; m.len_f = kv.len_target;
    m.n_rows_in = sc.n_rows; m.n_draft_in = sc.n_draft; m.tokens = sc.tokens; m.n_tokens = sc.n_tokens;
    m.tok_emb = (const __nv_bfloat16 *)c->tok_emb;
    if (a.mode == 1) m.h_src = (a.l0 == a.L_d) ? sc.hidden->h_draft : sc.hidden->h_inter;
    if (a.l1 == a.L_d) m.exit_buf = sc.hidden ? sc.hidden->h_draft : nullptr;
    else if (a.l1 == a.L_i) m.exit_buf = sc.hidden ? sc.hidden->h_inter : nullptr;
    m.hidden_out = sc.res ? sc.res->hidden_out : nullptr;
    m.k_pages = (__nv_bfloat16 *)kv.k_pages; m.v_pages = (__nv_bfloat16 *)kv.v_pages;
    m.block_table = kv.block_table; m.n_pages = kv.n_pages; m.first_layer = kv.first_layer;
    m.x = c->x; m.act_d = c->act_d; m.act_o = c->act_o; m.act_f = c->act_f; m.q = c->q; m.part = c->part;
    m.attn_part = c->attn_part; m.top_part = c->top_part; m.ssq = x->ssq; m.inv_freq = c->inv_freq; m.rope = x->rope; m.cta_top = x->cta_top;
    m.G = d.n_q_heads / d.n_kv_heads;
    const int QR = m.G * a.R_pad;
    m.n_mg = ceil_div(QR, 64);
    m.mt = ceil_div(QR < 64 ? QR : 64, 16);
    // one attention item per CTA where possible: the phase is latency-bound at small batch
    m.n_splits = c->sm_count / (a.batch * d.n_kv_heads * m.n_mg);
    {   // ... but long sequences still want about 64 pages per item
        int by_len = ceil_div(d.max_pages_per_seq, 64);
        if (m.n_splits < by_len) m.n_splits = by_len;
    }
    if (m.n_splits < 1) m.n_splits = 1;
    if (m.n_splits > 16) m.n_splits = 16;
    if ((long long)a.batch * d.n_kv_heads * m.n_mg * m.n_splits >= (1ll << 21)) return 1;   // attention item numbers, same rule
    m.ngrp = m.mt == 1 ? 4 : (m.mt == 2 ? 2 : 1);
    if (m.n_splits * m.ngrp > 32) m.ngrp = 32 / m.n_splits;   // one load batch in the split merge (16 splits: ngrp <= 2)
    if (m.ngrp == 3) m.ngrp = 2;
    m.attn_stages -= m.attn_stages % m.ngrp;   // a stage belongs to one warp group
    if (m.attn_stages < m.ngrp) return 1;
    if ((size_t)m.n_splits * m.ngrp * T_pad * d.n_q_heads * (d.head_dim + kAttnRecPad) > c->attn_part_floats) return 1;
    m.scale_log2 = (1.0f / sqrtf((float)d.head_dim)) * 1.4426950408889634f;
    m.r.len_d = kv.len_draft; m.r.len_i = kv.len_inter; m.r.len_f = kv.len_target;
    m.r.draft_tokens = sc.draft_tokens; m.r.token_stride = sc.token_stride; m.r.out_stride = sc.out_stride;
    if (sc.res) {
        m.r.n_accepted = sc.res->n_accepted; m.r.next_token = sc.res->next_token;
        m.r.argmax_ids = sc.res->argmax_ids; m.r.top2 = sc.res->top2; m.r.tentative = sc.res->tentative;
        m.r.pending = sc.res->pending;
        m.r.defer = sc.res->defer_accept;
        m.logits = sc.res->logits;
    }
    m.r.out_tokens = sc.out_tokens; m.r.n_tokens = sc.n_tokens;
    m.n_rep = sc.block ? sc.n_steps + (sc.bonus ? 1 : 0) : 1;
    m.block = sc.block; m.block_stride = sc.block_stride; m.n_steps = sc.n_steps;
    m.argmax_ws = c->argmax_ws;
    m.status = c->status;
    m.bar_count = x->bar + (x->bar_sel & 1); m.bar_next = x->bar + ((x->bar_sel + 1) & 1);
    x->bar_sel ^= 1;
    m.trace = x->trace;
    const CUtensorMap *tmd = act_map(c, 0, c->act_d, d.d_model, m.t_box, planes);
    const CUtensorMap *tmo = act_map(c, 1, c->act_o, d.n_q_heads * d.head_dim, m.t_box, planes);
    const CUtensorMap *tmf = act_map(c, 2, c->act_f, d.d_ffn, m.t_box, planes);
    const hispec_ctx_ext::PageMaps *pm = page_maps(c, kv);
    if (!tmd || !tmo || !tmf || !pm) return HISPEC_ECUDA;
    const size_t smem = (size_t)2 * stages * stage_bytes + attn_bytes + 1024;
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3(c->sm_count);
    cfg.blockDim = dim3(kMegaThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    c->launches++;
    double wbytes = 2.0 * (double)c->plan[G_HEAD].N * c->plan[G_HEAD].K;
    for (int k = 0; k < G_HEAD; ++k) wbytes += 2.0 * (double)c->plan[k].N * c->plan[k].K * (a.l1 - a.l0);
    wbytes *= m.n_rep;
    ProfScope prof(c, st, 20, wbytes);
    cudaError_t le = (d.head_dim == 64)
                         ? cudaLaunchKernelEx(&cfg, hispec_stage_kernel<64>, *tmd, *tmo, *tmf, pm->tmK, pm->tmV, m)
                         : cudaLaunchKernelEx(&cfg, hispec_stage_kernel<128>, *tmd, *tmo, *tmf, pm->tmK, pm->tmV, m);
    if (le == cudaErrorCooperativeLaunchTooLarge || le == cudaErrorLaunchOutOfResources) {
        // the GPU cannot hold one CTA per SM at once (e.g. it is shared): use the kernel sequence from now on
        (void)cudaGetLastError();
        x->mega_ok = false;
        x->bar_sel ^= 1;
        c->launches--;
        return 1;
    }
    CK(le);
    return HISPEC_OK;
}

int run_stage(hispec_ctx *c, cudaStream_t st, const StageCall &sc) {
    {
        int rc = run_stage_mega(c, st, sc);
        if (rc != 1) return rc;
    }
    const hispec_model_desc &d = c->d;
    const StageArgs &a = sc.a;
    hispec_ctx_ext *x = ext_of(c);
    const int T_pad = a.batch * a.R_pad;
    const int plain = (d.flags & HISPEC_FLAG_PLAIN_ACT) ? 1 : 0;
    const bool simt = (d.flags & HISPEC_FLAG_SIMT_GEMM) != 0;
    const hispec_kv &kv = *sc.kv;

    CK(launch(c, st, prep_rows_kernel, dim3(ceil_div(a.batch, 64)), dim3(64), 0, a, (const int32_t *)kv.len_draft,
              (const int32_t *)kv.len_inter, (const int32_t *)kv.len_target, sc.n_rows, sc.n_draft, sc.tokens,
              sc.n_tokens, c->rows, c->status));
    const float *h_src = nullptr;
    if (a.mode == 1) h_src = (a.l0 == a.L_d) ? sc.hidden->h_draft : sc.hidden->h_inter;
    CK(launch(c, st, rows_in_norm_kernel, dim3(T_pad), dim3(256), 0, a, c->rows, sc.tokens,
              (const __nv_bfloat16 *)c->tok_emb, d.vocab, h_src, c->attn_norm[a.l0], d.rms_eps, d.d_model, c->x,
              c->act_d, x->T_alloc, plain, c->status));

    float *exit_buf = nullptr;
    if (a.l1 == a.L_d) exit_buf = sc.hidden ? sc.hidden->h_draft : nullptr;
    else if (a.l1 == a.L_i) exit_buf = sc.hidden ? sc.hidden->h_inter : nullptr;
    float *hidden_out = sc.res ? sc.res->hidden_out : nullptr;

    for (int l = a.l0; l < a.l1; ++l) {
        const int pool_layer = l - kv.first_layer;
        int rc;
        const GemmPlan &pq = c->plan[G_QKV], &po = c->plan[G_O], &pg = c->plan[G_GU], &pd = c->plan[G_DOWN];
        int sq = pq.splits, so = po.splits, sg = pg.splits, sd = pd.splits;
        if ((rc = run_gemm(c, st, G_QKV, c->wqkv[l], &c->tm_wqkv[l], 0, T_pad, sc, &sq)) != 0) return rc;
        // a thread per rotary pair: four times the threads where a row has the pairs to fill them
        const int qk_threads = (d.n_q_heads + d.n_kv_heads) * (d.head_dim / 2) >= 1024 ? 1024 : 256;
        CK(launch(c, st, qkv_rope_store_kernel, dim3(T_pad), dim3(qk_threads), 0, a, c->rows, (const float *)c->part, sq,
                  (size_t)T_pad * pq.N, d.n_q_heads, d.n_kv_heads, d.head_dim, (const double *)c->inv_freq, c->q,
                  (__nv_bfloat16 *)kv.k_pages, (__nv_bfloat16 *)kv.v_pages, kv.block_table, (long long)kv.n_pages,
                  pool_layer, c->status));
        AttnArgs at;
        at.q = c->q; at.k_pages = (const __nv_bfloat16 *)kv.k_pages; at.v_pages = (const __nv_bfloat16 *)kv.v_pages;
        at.block_table = kv.block_table; at.n_pages = kv.n_pages; at.pool_layer = pool_layer;
        at.hq = d.n_q_heads; at.hkv = d.n_kv_heads; at.hd = d.head_dim;
        at.scale = 1.0f / sqrtf((float)d.head_dim);
        at.out = c->act_o; at.T_alloc = x->T_alloc; at.plain = plain;
        const bool tiled = d.page_size == 16 && !(d.flags & HISPEC_FLAG_ROWWARP_ATTN);
        if (!tiled) {
            ProfScope prof(c, st, 1, 0.0);
            int warps = T_pad * d.n_q_heads;
            dim3 grid(ceil_div(warps, 4));
            if (d.head_dim == 64) CK(launch(c, st, attention_rowwarp_kernel<64>, grid, dim3(128), 0, a, c->rows, at, c->status));
            else CK(launch(c, st, attention_rowwarp_kernel<128>, grid, dim3(128), 0, a, c->rows, at, c->status));
        } else {
            ProfScope prof(c, st, 1, 0.0);
            const hispec_ctx_ext::PageMaps *pm = page_maps(c, kv);
            if (!pm) return HISPEC_ECUDA;
            AttnTcArgs ta;
            ta.q = c->q; ta.block_table = kv.block_table; ta.n_pages = kv.n_pages; ta.pool_layer = pool_layer;
            ta.hq = d.n_q_heads; ta.hkv = d.n_kv_heads; ta.G = d.n_q_heads / d.n_kv_heads;
            const int QR = ta.G * a.R_pad;
            ta.n_mg = ceil_div(QR, kAttnGroupRows);
            ta.mt = ceil_div(QR < kAttnGroupRows ? QR : kAttnGroupRows, 16);
            ta.n_splits = attn_splits(c->sm_count, a.batch, d.n_kv_heads, ta.G, a.R_pad);
            ta.scale_log2 = at.scale * 1.4426950408889634f;
            ta.part = c->attn_part;
            if ((size_t)ta.n_splits * T_pad * d.n_q_heads * (d.head_dim + 2) > c->attn_part_floats) return HISPEC_ECAPACITY;
            dim3 grid(ta.n_splits, d.n_kv_heads * ta.n_mg, a.batch), block((ta.mt + 1) * 32);
            int mwarps = T_pad * d.n_q_heads;
            if (d.head_dim == 64) {
                CK(launch(c, st, attention_tc_kernel<64>, grid, block, 0, pm->tmK, pm->tmV, a, c->rows, ta, c->status));
                CK(launch(c, st, attention_merge_kernel<64>, dim3(ceil_div(mwarps, 4)), dim3(128), 0, a, c->rows,
                          (const float *)c->attn_part, ta.n_splits, d.n_q_heads, c->act_o, x->T_alloc, plain));
            } else {
                CK(launch(c, st, attention_tc_kernel<128>, grid, block, 0, pm->tmK, pm->tmV, a, c->rows, ta, c->status));
                CK(launch(c, st, attention_merge_kernel<128>, dim3(ceil_div(mwarps, 4)), dim3(128), 0, a, c->rows,
                          (const float *)c->attn_part, ta.n_splits, d.n_q_heads, c->act_o, x->T_alloc, plain));
            }
        }
        // one thread per four columns of the row, up to 1024 threads
        const int rn_threads = d.d_model / 4 >= 1024 ? 1024 : (d.d_model / 4 <= 64 ? 64 : round_up(d.d_model / 4, 32));
        if ((rc = run_gemm(c, st, G_O, c->wo[l], &c->tm_wo[l], 1, T_pad, sc, &so)) != 0) return rc;
        CK(launch(c, st, resid_norm_kernel, dim3(T_pad), dim3(rn_threads), 0, a, c->rows, (const float *)c->part, so,
                  (size_t)T_pad * po.N, c->ffn_norm[l], d.rms_eps, d.d_model, c->x, c->act_d, x->T_alloc, plain,
                  (float *)nullptr, (float *)nullptr));
        if ((rc = run_gemm(c, st, G_GU, c->wgu[l], &c->tm_wgu[l], 0, T_pad, sc, &sg)) != 0) return rc;
        CK(launch(c, st, silu_mul_kernel, dim3(ceil_div(d.d_ffn, 256), T_pad), dim3(256), 0, (const float *)c->part,
                  sg, (size_t)T_pad * pg.N, d.d_ffn, c->act_f, x->T_alloc, plain));
        if ((rc = run_gemm(c, st, G_DOWN, c->wdown[l], &c->tm_wdown[l], 2, T_pad, sc, &sd)) != 0) return rc;
        const bool last = (l + 1 == a.l1);
        const float *gain = last ? c->final_norm : c->attn_norm[l + 1];
        CK(launch(c, st, resid_norm_kernel, dim3(T_pad), dim3(rn_threads), 0, a, c->rows, (const float *)c->part, sd,
                  (size_t)T_pad * pd.N, gain, d.rms_eps, d.d_model, c->x, c->act_d, x->T_alloc, plain,
                  last ? exit_buf : (float *)nullptr, last ? hidden_out : (float *)nullptr));
    }
    const void *head = (a.l1 == a.L_d) ? sc.exits->head_d : ((a.l1 == a.L_i) ? sc.exits->head_i : sc.exits->head_f);
    const CUtensorMap *tmH = simt ? (const CUtensorMap *)c->tm_wqkv : head_map(c, head);
    int rc = run_gemm(c, st, G_HEAD, head, tmH, 0, T_pad, sc);
    if (rc) return rc;
    AcceptArgs r;
    memset(&r, 0, sizeof(r));
    r.len_d = kv.len_draft; r.len_i = kv.len_inter; r.len_f = kv.len_target;
    r.draft_tokens = sc.draft_tokens; r.token_stride = sc.token_stride; r.out_stride = sc.out_stride;
    if (sc.res) {
        r.n_accepted = sc.res->n_accepted; r.next_token = sc.res->next_token;
        r.argmax_ids = sc.res->argmax_ids; r.top2 = sc.res->top2; r.tentative = sc.res->tentative;
        r.pending = sc.res->pending;
        r.defer = sc.res->defer_accept;
    }
    r.out_tokens = sc.out_tokens;
    r.n_tokens = sc.n_tokens;
    int n_tiles = simt ? c->plan[G_HEAD].tiles : 4 * c->plan[G_HEAD].tiles;
    CK(launch(c, st, head_reduce_accept_kernel, dim3(a.batch), dim3(256), 0, a, c->rows, (const float *)c->top_part,
              n_tiles, T_pad, r, c->argmax_ws));
    return HISPEC_OK;
}

int check_common(hispec_ctx *c, int l0, int l1, const hispec_exits *ex, const hispec_kv *kv, int batch) {
    if (!c || !ex || !kv) return HISPEC_EINVAL;
    if (!(0 < ex->L_d && ex->L_d < ex->L_i && ex->L_i < ex->L_f && ex->L_f <= c->d.n_layers)) return HISPEC_EINVAL;
    if (l0 < 0 || l1 <= l0 || l1 > c->d.n_layers) return HISPEC_EINVAL;
    if (l1 != ex->L_d && l1 != ex->L_i && l1 != ex->L_f) return HISPEC_EINVAL;
    const void *head = (l1 == ex->L_d) ? ex->head_d : ((l1 == ex->L_i) ? ex->head_i : ex->head_f);
    if (!head) return HISPEC_EINVAL;
    if (batch <= 0) return HISPEC_EINVAL;
    if (batch > c->d.max_batch) return HISPEC_ECAPACITY;
    if (!kv->k_pages || !kv->v_pages || !kv->block_table || !kv->len_draft || !kv->len_inter || !kv->len_target ||
        kv->n_pages <= 0)
        return HISPEC_EINVAL;
    if (kv->first_layer < 0 || l0 < kv->first_layer || l1 > kv->first_layer + kv->n_pool_layers) return HISPEC_EINVAL;
    for (int l = l0; l < l1; ++l)
        if (!c->wqkv[l] || !c->wo[l] || !c->wgu[l] || !c->wdown[l] || !c->attn_norm[l] || !c->ffn_norm[l])
            return HISPEC_EINVAL;
    return HISPEC_OK;
}

StageArgs base_args(hispec_ctx *c, const hispec_exits *ex, int l0, int l1, int batch, int R_pad) {
    StageArgs a;
    memset(&a, 0, sizeof(a));
    a.L_d = ex->L_d; a.L_i = ex->L_i; a.L_f = ex->L_f; a.l0 = l0; a.l1 = l1;
    a.batch = batch; a.R_pad = R_pad; a.max_rows = c->d.max_rows_per_seq; a.max_pages = c->d.max_pages_per_seq;
    a.page_size = c->d.page_size;
    return a;
}

int verify_call(hispec_ctx *c, void *stream, int l0, int l1, const hispec_exits *ex, const hispec_kv *kv,
                const hispec_hidden *hid, int batch, const int32_t *draft_tokens, int token_stride,
                const int32_t *n_draft, const int32_t *n_rows, int k, const hispec_result *res, bool target) {
    int rc = check_common(c, l0, l1, ex, kv, batch);
    if (rc) return rc;
    if (!hid || !hid->h_draft || !hid->h_inter || !draft_tokens || !res || !res->n_accepted || !res->next_token)
        return HISPEC_EINVAL;
    if ((n_draft == nullptr) != (n_rows == nullptr)) return HISPEC_EINVAL;
    if (k < 0 || token_stride < k) return HISPEC_EINVAL;
    if (k + 1 > c->d.max_rows_per_seq) return HISPEC_ECAPACITY;
    if (target) {
        if (l0 != ex->L_i || l1 != ex->L_f) return HISPEC_EINVAL;
    } else {
        if (l0 != ex->L_d || (l1 != ex->L_i && l1 != ex->L_f)) return HISPEC_EINVAL;
    }
    StageCall sc;
    memset(&sc, 0, sizeof(sc));
    sc.a = base_args(c, ex, l0, l1, batch, k + 1);
    sc.a.mode = 1; sc.a.k = k; sc.a.is_target = target ? 1 : 0;
    sc.exits = ex; sc.kv = kv; sc.hidden = hid;
    sc.draft_tokens = draft_tokens; sc.n_draft = n_draft; sc.n_rows = n_rows; sc.token_stride = token_stride;
    sc.res = res;
    return run_stage(c, (cudaStream_t)stream, sc);
}

}  // namespace

extern "C" int hispec_draft(hispec_ctx *c, void *stream, int l0, int l1, const hispec_exits *ex, const hispec_kv *kv,
                            const hispec_hidden *hid, int batch, const int32_t *in_tokens, int in_stride,
                            int32_t *out_tokens, int out_stride, const hispec_result *res) {
    int rc = check_common(c, l0, l1, ex, kv, batch);
    if (rc) return rc;
    if (l0 != 0 || !in_tokens || in_stride < 1 || (out_tokens && out_stride < 1)) return HISPEC_EINVAL;
    if (l1 != ex->L_f && (!hid || !hid->h_draft || !hid->h_inter)) return HISPEC_EINVAL;
    StageCall sc;
    memset(&sc, 0, sizeof(sc));
    sc.a = base_args(c, ex, l0, l1, batch, 1);
    sc.a.mode = 0; sc.a.tok_stride = in_stride; sc.a.tok_offset = 0; sc.a.fixed_rows = 1;
    sc.exits = ex; sc.kv = kv; sc.hidden = hid; sc.tokens = in_tokens; sc.res = res; sc.out_tokens = out_tokens;
    sc.out_stride = out_stride;
    return run_stage(c, (cudaStream_t)stream, sc);
}

extern "C" int hispec_draft_block(hispec_ctx *c, void *stream, int l0, int l1, const hispec_exits *ex, const hispec_kv *kv,
                                  const hispec_hidden *hid, int batch, const int32_t *in_tokens, int in_stride,
                                  int32_t *block, int block_stride, int n_steps, int bonus, const hispec_result *res) {
    int rc = check_common(c, l0, l1, ex, kv, batch);
    if (rc) return rc;
    if (l0 != 0 || !in_tokens || in_stride < 1 || !block || n_steps < 1 || block_stride < n_steps) return HISPEC_EINVAL;
    if (l1 != ex->L_f && (!hid || !hid->h_draft || !hid->h_inter)) return HISPEC_EINVAL;
    if (l1 != ex->L_f && n_steps + (bonus ? 1 : 0) > c->d.max_rows_per_seq) return HISPEC_EINVAL;
    StageCall sc;
    memset(&sc, 0, sizeof(sc));
    sc.a = base_args(c, ex, l0, l1, batch, 1);
    sc.a.mode = 0; sc.a.tok_stride = in_stride; sc.a.tok_offset = 0; sc.a.fixed_rows = 1;
    sc.exits = ex; sc.kv = kv; sc.hidden = hid; sc.tokens = in_tokens; sc.res = res;
    sc.block = block; sc.block_stride = block_stride; sc.n_steps = n_steps; sc.bonus = bonus ? 1 : 0;
    if (!(c->d.flags & HISPEC_FLAG_MULTI_KERNEL)) {
        rc = run_stage_mega(c, (cudaStream_t)stream, sc);
        if (rc != 1) return rc;
    }
    // the persistent kernel does not take this call: the same steps as separate calls
    const int total = n_steps + (bonus ? 1 : 0);
    for (int s = 0; s < total; ++s) {
        rc = hispec_draft(c, stream, l0, l1, ex, kv, hid, batch, s == 0 ? in_tokens : block + (s - 1),
                          s == 0 ? in_stride : block_stride, s < n_steps ? block + s : nullptr, block_stride, res);
        if (rc) return rc;
    }
    return HISPEC_OK;
}

extern "C" int hispec_verify_intermediate(hispec_ctx *c, void *stream, int l0, int l1, const hispec_exits *ex,
                                          const hispec_kv *kv, const hispec_hidden *hid, int batch,
                                          const int32_t *draft_tokens, int token_stride, const int32_t *n_draft,
                                          const int32_t *n_rows, int k, const hispec_result *res) {
    return verify_call(c, stream, l0, l1, ex, kv, hid, batch, draft_tokens, token_stride, n_draft, n_rows, k, res, false);
}

extern "C" int hispec_verify_target(hispec_ctx *c, void *stream, int l0, int l1, const hispec_exits *ex,
                                    const hispec_kv *kv, const hispec_hidden *hid, int batch,
                                    const int32_t *draft_tokens, int token_stride, const int32_t *n_draft,
                                    const int32_t *n_rows, int k, const hispec_result *res) {
    return verify_call(c, stream, l0, l1, ex, kv, hid, batch, draft_tokens, token_stride, n_draft, n_rows, k, res, true);
}

extern "C" int hispec_prefill(hispec_ctx *c, void *stream, const hispec_exits *ex, const hispec_kv *kv, int batch,
                              const int32_t *tokens, const int32_t *n_tokens, int max_tokens, int32_t *first_token) {
    if (!ex) return HISPEC_EINVAL;
    int rc = check_common(c, 0, ex->L_f, ex, kv, batch);
    if (rc) return rc;
    if (!tokens || !n_tokens || max_tokens <= 0) return HISPEC_EINVAL;
    const int C = c->d.max_rows_per_seq;
    for (int off = 0; off < max_tokens; off += C) {
        StageCall sc;
        memset(&sc, 0, sizeof(sc));
        sc.a = base_args(c, ex, 0, ex->L_f, batch, C);
        sc.a.mode = 0; sc.a.tok_stride = max_tokens; sc.a.tok_offset = off;
        sc.exits = ex; sc.kv = kv; sc.tokens = tokens; sc.n_tokens = n_tokens; sc.out_tokens = first_token;
        sc.out_stride = 1;
        rc = run_stage(c, (cudaStream_t)stream, sc);
        if (rc) return rc;
    }
    return HISPEC_OK;
}
