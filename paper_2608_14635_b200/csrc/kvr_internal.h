// Internal declarations shared by the host orchestration and the kernel files.
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <cuda.h>
#include <stdint.h>
#include <vector>

#include "kvrebuild.h"

namespace kvr {

// Arena addressing: element index of (layer, kv, flat slot, head 0, dim 0).
struct ArenaView {
    void *base;
    int64_t kv_stride;     // elements between K and V planes of a layer = NB * B * row
    int64_t layer_stride;  // elements per layer = 2 * kv_stride
    int32_t row;           // elements per token row = Hkv * hd
    int32_t block_size, num_blocks, n_kv_heads, head_dim;
};

struct ModelDims {
    int32_t L, d, Hq, Hkv, hd, F, V;
    int32_t q_dim, kv_dim;
    float eps;
    double rope_base;
};

// Per-chunk device metadata (all int32, n = tokens in the chunk).
struct ChunkMeta {
    const int32_t *tok;    // token id
    const int32_t *pos;    // position in its request's prefix
    const int32_t *slot;   // flat arena slot
    const int32_t *trow;   // row of the request in the device block-table array
    int32_t n;
};

// Attention work item for the tensor-core kernel: one tile of query rows of
// one request segment.
struct AttnTile {
    int32_t q_off;     // chunk-local index of the tile's first query token
    int32_t pos0;      // prefix position of that token
    int32_t rows;      // query rows in this tile (<= tile size)
    int32_t trow;      // block-table row
};

struct RopeFreq {
    double inv_freq[64];  // base^(-2i/hd), i < hd/2 <= 64
};

#ifdef __CUDACC__
// Programmatic dependent launch: a kernel launched with `pdl` may be scheduled while the kernel before it on
// the stream is still draining; it must not touch global memory before grid_dependency_wait(), which returns
// once that kernel has completed and its writes are visible (at once when the launch was an ordinary one).
// Every thread of every block calls it, so a kernel's completion implies the completion of all before it.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
// Lets the next kernel's blocks be scheduled as soon as all of this kernel's blocks have said so or exited.
__device__ __forceinline__ void grid_launch_dependents() {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, bool pdl,
                                 Args &&...args) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = pdl ? 1 : 0;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#endif

// ---- plain-FMA kernels (kvr_simt.cu); T selected by `fp32` ----
void launch_embed_rmsnorm(bool fp32, const void *embed, const void *gain, const ChunkMeta &cm, float *h,
                          void *a, int d, float eps, cudaStream_t s);
void launch_rmsnorm(bool fp32, const float *h, const void *gain, void *a, int n, int d, float eps,
                    cudaStream_t s);
// h_out = h_in + part[0] + ... + part[n_part - 1] (all fp32 [n, d], partial products part_stride elements apart;
// h_out may be h_in), then a = rmsnorm(h_out) * gain: the residual add of a row-parallel projection's partial
// sums folded into the norm that follows it
void launch_add_rmsnorm(bool fp32, const float *h_in, float *h_out, const float *part, int n_part,
                        int64_t part_stride, const void *gain, void *a, int n, int d, float eps, cudaStream_t s,
                        bool pdl = false);
void launch_rope_table(const int32_t *pos, int n, int hd, const RopeFreq &f, float2 *cs, cudaStream_t s);
// mode 0: C fp32 [M, ldc] = A W0^T; 1: C fp32 += A W0^T; 2: C (T) = silu(A W0^T) * (A W1^T)
void launch_gemm_simt(bool fp32, int mode, const void *A, int lda, const void *W0, const void *W1, int ldw,
                      int M, int N, int K, void *C, int ldc, cudaStream_t s);
// Optional terms of the q/k/v projections of one layer (device pointers in the model's
// element type, null = absent): biases [q_dim], [kv_dim], [kv_dim] and per-head RMSNorm
// gains [hd] applied to q and k after the bias and before RoPE.
struct QkvExtras {
    const void *bq = nullptr, *bk = nullptr, *bv = nullptr, *qn = nullptr, *kn = nullptr;
    float eps = 0.f;
    bool any() const { return bq || bk || bv || qn || kn; }
};
// Reads raw fp32 [n, q_dim + 2 kv_dim] projections (the sum of n_part partial products part_stride
// elements apart); writes rotated Q (T) and the arena rows.
void launch_rope_scatter(bool fp32, const float *qkv, int ld, const float2 *cs, const ChunkMeta &cm,
                         const ModelDims &md, const ArenaView &av, int layer, bool want_q, void *q_out,
                         const QkvExtras &ex, cudaStream_t s, int n_part = 1, int64_t part_stride = 0,
                         bool pdl = false);
void launch_attn_simt(bool fp32, const void *q, const ChunkMeta &cm, const int32_t *tables, int max_blk,
                      const ModelDims &md, const ArenaView &av, int layer, void *o, cudaStream_t s);
void launch_gather_rows(const float *h, int d, const int2 *pairs, int n_pairs, float *h_last, cudaStream_t s);
void launch_readback(bool fp32, const ArenaView &av, int layer, const int32_t *table_dev, int n, void *k_out,
                     void *v_out, cudaStream_t s);

// ---- tcgen05 GEMM (kvr_gemm_tc.cu) ----
struct TcGemmEpilogue {
    int mode;               // see TC_* below
    int M, N, K;            // N = logical output columns over all B operands
    // plain / residual
    float *c_f32;           // TC_STORE_F32, TC_RESID
    int ldc;
    // SwiGLU
    __nv_bfloat16 *out_bf16;  // TC_SWIGLU: [M, N/2]
    int ld_out;
    // QKV + RoPE + paged store
    __nv_bfloat16 *q_out;   // [M, q_dim]
    const float2 *rope_cs;  // [M, hd/2]
    const int32_t *slot;    // [M]
    __nv_bfloat16 *arena_k; // layer's K plane base; V plane = arena_k + kv_stride
    int64_t kv_stride;
    int n_q_cols, n_kv_cols, head_dim;
    const __nv_bfloat16 *bias_q, *bias_k, *bias_v;   // optional (null = none)
    const __nv_bfloat16 *gain_q, *gain_k;            // optional per-head RMSNorm gains [head_dim]
    float qk_eps;
    int resid_tma;          // TC_RESID: add through a TMA reduce (set by the launcher)
    int n_b;                // number of B operands in use (1..3)
    int b_rows[3];          // rows (output features) of each B operand
};
enum { TC_STORE_F32 = 0, TC_RESID = 1, TC_SWIGLU = 2, TC_QKV = 3 };

int tc_gemm_init(int device);  // driver entry points, kernel attributes; returns kvr_status
int tc_make_tmap_2d(CUtensorMap *out, const void *base, int64_t rows, int64_t cols, int box_rows, int box_cols);
int tc_make_tmap_kv(CUtensorMap *out, const void *base, int64_t rows, int64_t cols, int halves);
int tc_make_tmap_f32(CUtensorMap *out, const void *base, int64_t rows, int64_t cols);
// tmH: fp32 map over the residual (TC_RESID only); null = plain read-modify-write epilogue
// pair: run on CTA pairs (256 x 256 tiles, tcgen05 cta_group::2) instead of single CTAs
int launch_gemm_tc(const CUtensorMap &tmA, const CUtensorMap *tmB /*[3]*/, const TcGemmEpilogue &ep,
                   int *d_status, int n_sms, cudaStream_t s, const CUtensorMap *tmH = nullptr, bool pair = false);

// ---- weight-streaming GEMM for the few rows of kv_resume_logits (kvr_gemm_skinny.cu) ----
constexpr int GEMM_SKINNY_MAX_ROWS = 128, GEMM_SKINNY_MAX_SPLITS = 8;
struct SkinnyArgs {
    int R, N, K;              // out[r, n] = sum_k X[r, k] W[n, k], r < R <= 128
    float *out_f32;           // plain: partial product of split s at out_f32 + s * split_stride, row stride ldo
    int64_t split_stride;
    int ldo;
    __nv_bfloat16 *out_bf16;  // SwiGLU pair (two weight maps): silu(X Wg^T) * (X Wu^T), row stride ld_bf16
    int ld_bf16;
};
int gemm_skinny_init(int device);
int gemm_skinny_splits(int N, int K, int n_sms);
// tmX: activation map (box x_rows x 64, x_rows = 64 or 128), tmW0 / tmW1: weight maps (box 128 x 64);
// tmW1 non-null = SwiGLU pair
int launch_gemm_skinny(const CUtensorMap &tmX, const CUtensorMap &tmW0, const CUtensorMap *tmW1,
                       const SkinnyArgs &a, int x_rows, int splits, int *d_status, int n_sms, cudaStream_t s,
                       bool pdl = false);

// ---- tensor-core attention (kvr_attn_tc.cu) ----
int attn_tc_init(int device);
int launch_attn_tc(const __nv_bfloat16 *q, const AttnTile *tiles, int n_tiles, const int32_t *tables, int max_blk,
                   const ModelDims &md, const ArenaView &av, int layer, __nv_bfloat16 *o, int *d_status,
                   cudaStream_t s);
constexpr int ATTN_TILE_Q = 64;

// ---- tcgen05 attention (kvr_attn_fa.cu): tiles of up to 256 query rows ----
constexpr int ATTN_FA_TILE_Q = 256;
int attn_fa_init(int device);
int launch_attn_fa(const CUtensorMap &tmQ, const CUtensorMap &tmKV, const AttnTile *tiles, int n_tiles,
                   const int32_t *tables, int max_blk, const ModelDims &md, const ArenaView &av, int layer,
                   __nv_bfloat16 *o, int *d_status, cudaStream_t s);

// ---- single-row attention for resume logits (kvr_attn_decode.cu): split-KV, one pass over the request's K/V ----
constexpr int ATTN_DECODE_MAX_SPLITS = 16;
size_t attn_decode_scratch_bytes(int max_requests, int Hq, int hd);
// q [R, Hq*hd] bf16, pos[r] = position of the query row (it attends to keys 0..pos[r]); max_len = max(pos) + 1
int launch_attn_decode(const __nv_bfloat16 *q, const int32_t *pos, int R, int max_len, const int32_t *tables,
                       int max_blk, const ModelDims &md, const ArenaView &av, int layer, float *scratch,
                       __nv_bfloat16 *o, cudaStream_t s, bool pdl = false);

// ---- handover device steps (kvr_handover.cu) ----
constexpr int PROBE_THREADS = 64, PROBE_ITERS = 1000, PROBE_MAX_BLOCKS = 1024;
int launch_arena_flush(void *arena, size_t bytes, uint32_t word, int n_sms, cudaStream_t s);
int launch_probe(uint32_t seed, uint32_t epoch, uint32_t *flags, uint32_t *out, int *status, int blocks,
                 long long limit_cycles, int publish, cudaStream_t s);

}  // namespace kvr
