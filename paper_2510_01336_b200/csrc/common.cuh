// Shared declarations of the HiSpec CUDA library (sm_100a only).
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/hispec.h"

namespace hispec {

constexpr int kWeightTileRows = 128;  // output features per GEMM tile (UMMA M)
constexpr int kTileK = 64;            // bf16 elements per 128-byte swizzle row
constexpr int kMaxGemmRows = 256;     // activation rows one GEMM launch can take
constexpr int kMaxSplits = 16;
constexpr int kAttnMaxRows = 32;      // rows per sequence per call the attention kernel supports

enum GemmKind { G_QKV = 0, G_O = 1, G_GU = 2, G_DOWN = 3, G_HEAD = 4, G_KINDS = 5 };

struct GemmPlan {
    int N, K;        // output features, reduction length
    int tiles;       // ceil(N / 128)
    int splits;      // split-K factor
    int kb_total;    // ceil(K / 64) k-blocks
};

// Per-call row bookkeeping, filled on the device by prep_rows_kernel.
struct RowMeta {
    int32_t *p0;       // [max_batch] position of row 0
    int32_t *n_rows;   // [max_batch] valid rows
    int32_t *n_draft;  // [max_batch]
    int32_t *dst_row;  // [max_batch] first destination row in the exit buffer
};

}  // namespace hispec

struct hispec_ctx {
    hispec_model_desc d;
    int device;
    int sm_count;
    // pointer tables (host copies)
    const void *tok_emb;
    const void **wqkv, **wo, **wgu, **wdown;
    const float **attn_norm, **ffn_norm;
    const float *final_norm;
    // TMA descriptors, host side; one per weight matrix (+ heads created lazily)
    CUtensorMap *tm_wqkv, *tm_wo, *tm_wgu, *tm_wdown;
    struct HeadMap { const void *ptr; CUtensorMap map; } head_maps[4];
    int n_head_maps;
    CUtensorMap tm_act_d, tm_act_o, tm_act_f;  // activation operands [2][T_max][K]
    // workspace (device)
    int T_max;            // max_batch * max_rows_per_seq
    float *x;             // [T_max][d] residual stream
    __nv_bfloat16 *act_d; // [2][T_max][d]        normed rows (hi plane, lo plane)
    __nv_bfloat16 *act_o; // [2][T_max][hq*hd]    attention output
    __nv_bfloat16 *act_f; // [2][T_max][ffn]      SwiGLU activations
    float *q;             // [T_max][hq*hd] rotated queries
    float *part;          // split-K partial sums [splits][T_pad][N]
    size_t part_floats;
    float *attn_part;     // [T_max][hq][splits][hd + 2]
    int attn_max_splits;
    size_t attn_part_floats;
    float *top_part;      // [vocab tiles][T_max][4]: v1, id1, v2, pad
    float *logits_ws;     // [kMaxGemmRows][vocab], SIMT debug path only
    double *inv_freq;     // [hd/2] rotary frequencies
    hispec::RowMeta rows;
    int32_t *argmax_ws;   // [T_max]
    float *top2_ws;       // [T_max][2]
    uint32_t *status;     // device status word
    hispec::GemmPlan plan[hispec::G_KINDS];
    int64_t launches;
};
