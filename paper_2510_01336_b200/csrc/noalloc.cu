// hispec_exit_argmax_noalloc: exit head + greedy token for a few hidden rows without any
// allocation.
//
// Who needs this: a caller that has no way to obtain device memory at the moment it wants an
// exit's verdict -- a serving process that handed all free HBM to its KV-page pool at start-up
// (so cudaMalloc would fail or stall on a synchronising free), a thread that runs while
// another thread holds the allocator, or a plug-in that is only given raw pointers and a
// stream and is forbidden to touch the allocator of its host program.  Such a caller cannot
// create an hispec context either (hispec_create allocates its workspace), so this entry point
// works without one.
//
// The scratch the computation needs (normalised rows and per-tile top-2 records) lives in one
// file-scope __device__ array of fixed size.  Every GPU that loads the library carries that
// array (1 MiB) until the process exits.  All calls share it and it keeps whatever the last
// call left there; each call overwrites every element it later reads, so nothing has to be
// cleared, but two calls whose kernels overlap on the GPU (different streams, no ordering)
// race on it and give undefined results.  Order such calls yourself.
//
// In host code the array's name is only a stand-in for the device symbol, not a device
// address.  Its address is fetched once per device, with that device current, by
// cudaGetSymbolAddress during the first call on that device; that first call should therefore
// happen before any stream capture begins.
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include "../../include/hispec.h"

namespace {

constexpr int kRows = HISPEC_NOALLOC_MAX_ROWS;
constexpr int kMaxD = HISPEC_NOALLOC_MAX_D;
constexpr int kMaxVocab = HISPEC_NOALLOC_MAX_VOCAB;
constexpr int kTile = 128;                      // vocabulary entries per block
constexpr int kMaxTiles = kMaxVocab / kTile;
constexpr size_t kNormFloats = (size_t)kRows * kMaxD;
constexpr size_t kRecFloats = (size_t)kMaxTiles * kRows * 4;

static __device__ __align__(256) float g_scratch[kNormFloats + kRecFloats];

// device address of g_scratch per device ordinal, filled on first use
static float *g_scratch_addr[64] = {nullptr};

struct Rec {
    float v1, v2;
    int i1;
};
__device__ __forceinline__ Rec rec_merge(Rec a, Rec b) {  // larger value first, lower id on a tie
    bool a_first = (a.v1 > b.v1) || (a.v1 == b.v1 && a.i1 <= b.i1);
    Rec r;
    if (a_first) { r.v1 = a.v1; r.i1 = a.i1; r.v2 = fmaxf(a.v2, b.v1); }
    else { r.v1 = b.v1; r.i1 = b.i1; r.v2 = fmaxf(b.v2, a.v1); }
    return r;
}

// normed[t][i] = x[t][i] / sqrt(mean(x[t]^2) + eps) * gain[i]
__global__ void na_norm_kernel(const float *hidden, const float *gain, float eps, int d, float *normed) {
    __shared__ float red[32];
    const int t = blockIdx.x;
    const float *x = hidden + (size_t)t * d;
    float ss = 0.f;
    for (int i = threadIdx.x; i < d; i += blockDim.x) ss += x[i] * x[i];
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
    __syncthreads();
    float tot = 0.f;
    for (int i = 0; i < (int)(blockDim.x >> 5); ++i) tot += red[i];
    const float inv = rsqrtf(tot / (float)d + eps);
    for (int i = threadIdx.x; i < d; i += blockDim.x) normed[(size_t)t * kMaxD + i] = x[i] * inv * gain[i];
}

// one block per 128 vocabulary entries: logits of all rows, reduced to a top-2 record per row
__global__ void na_head_tile_kernel(const __nv_bfloat16 *head, const float *normed, int d, int vocab, int n_rows,
                                    float *recs) {
    __shared__ float s_v1[8][kRows], s_v2[8][kRows];
    __shared__ int s_i1[8][kRows];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int tile = blockIdx.x;
    Rec best[kRows];
#pragma unroll
    for (int t = 0; t < kRows; ++t) best[t] = Rec{-INFINITY, -INFINITY, 0x7fffffff};
    for (int r = 0; r < kTile / 8; ++r) {
        const int n = tile * kTile + warp * (kTile / 8) + r;
        if (n >= vocab) break;  // uniform across the warp
        const __nv_bfloat16 *w = head + (size_t)n * d;
        float acc[kRows];
#pragma unroll
        for (int t = 0; t < kRows; ++t) acc[t] = 0.f;
        for (int k = lane; k < d; k += 32) {
            const float wv = __bfloat162float(w[k]);
#pragma unroll
            for (int t = 0; t < kRows; ++t)
                if (t < n_rows) acc[t] += wv * normed[(size_t)t * kMaxD + k];
        }
#pragma unroll
        for (int t = 0; t < kRows; ++t) {
            float v = acc[t];
            for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
            best[t] = rec_merge(best[t], Rec{v, -INFINITY, n});
        }
    }
    if (lane == 0)
        for (int t = 0; t < kRows; ++t) { s_v1[warp][t] = best[t].v1; s_v2[warp][t] = best[t].v2; s_i1[warp][t] = best[t].i1; }
    __syncthreads();
    if (threadIdx.x < n_rows) {
        const int t = threadIdx.x;
        Rec m = Rec{s_v1[0][t], s_v2[0][t], s_i1[0][t]};
        for (int w = 1; w < 8; ++w) m = rec_merge(m, Rec{s_v1[w][t], s_v2[w][t], s_i1[w][t]});
        float *o = recs + ((size_t)tile * kRows + t) * 4;
        o[0] = m.v1; o[1] = __int_as_float(m.i1); o[2] = m.v2;
    }
}

// one block per row: combine the tile records in tile order
__global__ void na_reduce_kernel(const float *recs, int n_tiles, int32_t *argmax_ids, float *top2) {
    __shared__ float s_v1[32], s_v2[32];
    __shared__ int s_i1[32];
    const int t = blockIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    Rec best = Rec{-INFINITY, -INFINITY, 0x7fffffff};
    for (int tile = threadIdx.x; tile < n_tiles; tile += blockDim.x) {
        const float *o = recs + ((size_t)tile * kRows + t) * 4;
        best = rec_merge(best, Rec{o[0], o[2], __float_as_int(o[1])});
    }
    for (int o = 16; o > 0; o >>= 1) {
        Rec other;
        other.v1 = __shfl_xor_sync(0xffffffffu, best.v1, o);
        other.v2 = __shfl_xor_sync(0xffffffffu, best.v2, o);
        other.i1 = __shfl_xor_sync(0xffffffffu, best.i1, o);
        best = rec_merge(best, other);
    }
    if (lane == 0) { s_v1[warp] = best.v1; s_v2[warp] = best.v2; s_i1[warp] = best.i1; }
    __syncthreads();
    if (threadIdx.x == 0) {
        Rec m = Rec{s_v1[0], s_v2[0], s_i1[0]};
        for (int w = 1; w < (int)(blockDim.x >> 5); ++w) m = rec_merge(m, Rec{s_v1[w], s_v2[w], s_i1[w]});
        argmax_ids[t] = m.i1;
        if (top2) { top2[2 * t] = m.v1; top2[2 * t + 1] = m.v2; }
    }
}

}  // namespace

extern "C" int hispec_exit_argmax_noalloc(void *stream, const void *head, const float *final_norm, float rms_eps,
                                          int d_model, int vocab, const float *hidden, int n_rows,
                                          int32_t *argmax_ids, float *top2) {
    if (!head || !final_norm || !hidden || !argmax_ids || d_model <= 0 || vocab <= 0 || n_rows <= 0) return HISPEC_EINVAL;
    if (n_rows > kRows || d_model > kMaxD || vocab > kMaxVocab) return HISPEC_ECAPACITY;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return HISPEC_ECUDA;
    if (!g_scratch_addr[dev]) {  // set-up, once per device, with that device current
        float *p = nullptr;
        if (cudaGetSymbolAddress((void **)&p, g_scratch) != cudaSuccess || !p) return HISPEC_ECUDA;
        g_scratch_addr[dev] = p;
    }
    float *normed = g_scratch_addr[dev];
    float *recs = normed + kNormFloats;
    cudaStream_t st = (cudaStream_t)stream;
    const int tiles = (vocab + kTile - 1) / kTile;
    na_norm_kernel<<<n_rows, 256, 0, st>>>(hidden, final_norm, rms_eps, d_model, normed);
    na_head_tile_kernel<<<tiles, 256, 0, st>>>((const __nv_bfloat16 *)head, normed, d_model, vocab, n_rows, recs);
    na_reduce_kernel<<<n_rows, 256, 0, st>>>(recs, tiles, argmax_ids, top2);
    return cudaGetLastError() == cudaSuccess ? HISPEC_OK : HISPEC_ECUDA;
}
