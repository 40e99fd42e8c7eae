/*
 * kvrebuild — rebuild request K/V in a retained paged KV arena from logged
 * token prefixes (sm_100a, one GPU).
 *
 * Operation: after a rollout worker fails, the replacement worker keeps the
 * independently owned weights and raw KV-cache pool, flushes the pool, and
 * reconstructs each interrupted request's K/V by prefilling the token prefix
 * the router logged for it (paper Sec. 4.1 "State isolation", Sec. 4.2
 * handover steps 2 and 5, Sec. 4.3 token-level context recovery).  This
 * library is that prefill: a batched, variable-length causal forward of a
 * pre-norm decoder (RMSNorm, grouped-query attention, rotate-half RoPE,
 * SwiGLU, no biases) whose K (after RoPE) and V rows are written into arena
 * blocks through per-request block tables.
 *
 * Conventions for every call
 *   - Returns a kvr_status (0 = KVR_OK, negative = error).  No exceptions, no
 *     abort, no device traps.  A call that fails validation enqueues nothing
 *     and leaves the arena byte-identical.
 *   - "dev" pointers are device memory of the context's GPU, "host" pointers
 *     are ordinary host memory.  The library never frees or reallocates memory
 *     the caller passes in, and keeps no reference to host arrays after the
 *     call returns.
 *   - One context per device; calls on one context must not overlap in time
 *     (the caller serialises them).
 *   - Streams are passed as `void *` holding a cudaStream_t (NULL = default).
 *
 * Arena layout (element type = geometry.dtype, base 256-byte aligned):
 *     arena[layer][0=K,1=V][block][slot][kv_head][dim]
 * Token t of a request lives in block table[t / block_size], slot
 * t % block_size, in every layer.
 */
#ifndef KVREBUILD_H
#define KVREBUILD_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct kvr_ctx kvr_ctx; /* opaque; one per device */

typedef enum {
    KVR_OK = 0,
    KVR_ERR_INVALID_ARG = -1,     /* null pointer, negative size, inconsistent geometry */
    KVR_ERR_NOT_BOUND = -2,       /* arena, weights or workspace not bound yet */
    KVR_ERR_UNSUPPORTED = -3,     /* shape outside what the kernels implement */
    KVR_ERR_BLOCK_OOB = -4,       /* block id outside [0, num_blocks) */
    KVR_ERR_TABLE_TOO_SHORT = -5, /* fewer valid table entries than ceil(len / block_size) */
    KVR_ERR_ALIAS_CONFLICT = -6,  /* one block at two logical positions or under different tokens */
    KVR_ERR_TOKEN_OOB = -7,       /* token id outside [0, vocab) */
    KVR_ERR_WORKSPACE = -8,       /* workspace too small for this call */
    KVR_ERR_CUDA = -9,            /* a CUDA runtime/driver call failed */
    KVR_ERR_DEVICE_TIMEOUT = -10  /* a bounded device-side wait expired (kv_sync_status) */
} kvr_status;

typedef enum { KVR_BF16 = 0, KVR_FP32 = 1 } kvr_dtype;

/* Decoder shape.  dtype is the type of weights, activations and arena; fp32 is
 * a correctness mode (plain FMA kernels), bf16 the production mode. */
typedef struct {
    int32_t n_layers, d_model, n_q_heads, n_kv_heads, head_dim, ffn, vocab;
    float rms_eps, rope_base;
    int32_t dtype; /* kvr_dtype */
} kv_model_desc;

typedef struct {
    int32_t block_size, num_blocks, n_layers, n_kv_heads, head_dim;
    int32_t dtype; /* kvr_dtype */
} kv_arena_geometry;

/* Device pointers to the weights.  Linear weights are [out, in] row-major;
 * gains are [d_model].  Each of the nine arrays is a HOST array of n_layers
 * device pointers. */
typedef struct {
    const void *embed; /* dev [vocab, d_model] */
    const void *const *ln1, *const *wq, *const *wk, *const *wv, *const *wo;
    const void *const *ln2, *const *wg, *const *wu, *const *wd;
} kv_weights;

/* Create / destroy a context on CUDA device `device`.  Creation allocates only
 * a few KB of pinned host memory and one device status word. */
int kv_ctx_create(kvr_ctx **out, int device);
int kv_ctx_destroy(kvr_ctx *ctx);

/* Paper Sec. 4.1 / Sec. 5: the worker obtains the KV-cache pool's pointer and
 * metadata from its owner.  `arena_dev` stays caller-owned; arena_bytes must
 * cover n_layers * 2 * num_blocks * block_size * n_kv_heads * head_dim
 * elements.  Nothing is written. */
int kv_arena_bind(kvr_ctx *ctx, void *arena_dev, size_t arena_bytes, const kv_arena_geometry *geom);

/* Paper Sec. 4.1: weights live under an independent owner and are reused in
 * place.  The pointer arrays are copied; the weights themselves are neither
 * copied nor modified (tensor maps over them are built here). */
int kv_weights_bind(kvr_ctx *ctx, const kv_model_desc *desc, const kv_weights *weights);

/* Paper Sec. 6 (models): the end-to-end runs use a family whose attention applies a
 * per-head RMSNorm to q and k before RoPE, the re-prefill figure one whose q/k/v
 * projections carry biases.  Both are optional terms of the projection step:
 *   bq, bk, bv       host arrays of n_layers device pointers, [q_dim], [kv_dim], [kv_dim]
 *                    (all three or none): q = Wq a + bq, ...
 *   q_norm, k_norm   host arrays of n_layers device pointers to gains [head_dim] (both
 *                    or none): every q and k head row x becomes
 *                    x / sqrt(mean(x^2) + rms_eps) * gain, after the bias, before RoPE.
 * Elements have the model dtype, pointers are 16-byte aligned and stay caller-owned.
 * Call after kv_weights_bind (which clears the variant); NULL clears it.  Applies to
 * kv_rebuild, kv_rebuild_from and kv_resume_logits alike. */
typedef struct {
    const void *const *bq, *const *bk, *const *bv;
    const void *const *q_norm, *const *k_norm;
} kv_proj_variant;
int kv_variant_bind(kvr_ctx *ctx, const kv_proj_variant *variant);

/* Paper Sec. 6.1 (experimental setup): the rollout engines whose KV is rebuilt are tensor-parallel
 * (TP = 2 / 4).  Under TP every rank holds the whole residual stream, its own share of the
 * attention heads and of the SwiGLU columns, and its own KV pool with its share of the kv heads;
 * the two row-parallel products of a layer (output projection, down projection) yield partial
 * sums that are added over the ranks before they enter the residual.
 *
 * A context runs one rank.  The shapes it is bound with are the rank's LOCAL ones
 * (kv_tp_plan_host gives them): n_q_heads, n_kv_heads and ffn are per-rank counts, d_model and
 * vocab are whole; weights are the rank's slices (wq/wk/wv/wg/wu: a range of rows, wo/wd: a range
 * of columns, as contiguous matrices of the local shape; norms and embedding whole); the arena is
 * the rank's pool (n_kv_heads local).  kv_tp_bind then names the exchange step:
 *   allreduce(buf_dev, count, stream, user) must enqueue on `stream` an in-place sum over all
 *   ranks of `count` fp32 values at buf_dev (device memory of this rank) and return 0, or return
 *   non-zero on failure (kv_rebuild then returns KVR_ERR_CUDA).  It is called on the host, inside
 *   kv_rebuild, twice per layer and chunk, in the same order on every rank; the library itself
 *   contains no collective and never touches another rank's memory.
 * tp_world = 1 (or config NULL) clears the sharding.  Call after kv_weights_bind and before
 * kv_workspace_bytes / kv_workspace_bind (the workspace gains one fp32 [chunk, d_model] buffer).
 * All ranks must be given the same batch, chunk size and options.  kv_resume_logits works under TP
 * too: every rank finishes the last layer with its slices, calls the callback twice (after the output
 * and the down projection, on up to 8 * R * d_model values) and multiplies by the whole LM head, so
 * every rank ends with the same logits. */
typedef int (*kv_allreduce_fn)(void *buf_dev, int64_t count, void *stream, void *user);
typedef struct {
    int32_t tp_world, tp_rank;
    kv_allreduce_fn allreduce;
    void *user;
} kv_tp_config;
int kv_tp_bind(kvr_ctx *ctx, const kv_tp_config *config);

/* Host-only partition plan of a model over tp_world ranks (needs no GPU and no context): rank r
 * takes q heads [q_head0, q_head0 + n_q_heads), kv heads [kv_head0, ...) -- whole GQA groups, so a
 * rank's q heads only ever read its own kv heads -- and SwiGLU columns [ffn0, ffn0 + ffn).
 * local_out receives the descriptor to bind on that rank.  KVR_ERR_UNSUPPORTED if tp_world does
 * not divide n_kv_heads and ffn / 8. */
typedef struct {
    int32_t q_head0, n_q_heads, kv_head0, n_kv_heads, ffn0, ffn;
} kv_tp_shard;
int kv_tp_plan_host(const kv_model_desc *full, int32_t tp_world, int32_t tp_rank, kv_model_desc *local_out,
                    kv_tp_shard *shard_out);

/* Scratch the rebuild needs for chunks of at most max_chunk_tokens tokens,
 * batches of at most max_requests requests and tables of at most
 * max_blocks_per_req entries.  Needs the weights bound (for the shape).
 * Returns 0 on error.  The workspace is caller-owned device memory,
 * 256-byte aligned; kv_rebuild allocates nothing on the device. */
size_t kv_workspace_bytes(const kvr_ctx *ctx, int64_t max_chunk_tokens, int32_t max_requests,
                          int32_t max_blocks_per_req);
int kv_workspace_bind(kvr_ctx *ctx, void *ws_dev, size_t ws_bytes, int64_t max_chunk_tokens,
                      int32_t max_requests, int32_t max_blocks_per_req);

/* Paper Sec. 4.2 step 5 + Sec. 4.3: rebuild the K/V of n_requests logged
 * prefixes into the bound arena.
 *   weights         NULL = the bound set (the only supported value besides the
 *                   same pointers again)
 *   token_prefixes  host int32 [sum(prefix_lens)], request after request
 *   prefix_lens     host int32 [n_requests]; 0 is a valid no-op request
 *   block_tables    host int32 [n_requests][max_blocks_per_req], -1 padded
 * Validates everything on the host first (order: lengths, table coverage,
 * block range, token range, aliasing), then enqueues the work on `stream` and
 * returns without waiting.  The arena rows slot(r, t) of every layer hold the
 * request's K/V once the stream reaches that point; no other arena byte is
 * written (slots past a prefix's end in its last block keep their bytes).
 * Requests that share leading full blocks (same block ids, same tokens) have
 * those blocks computed and written once.  Rebuilding twice gives bit-identical
 * results. */
int kv_rebuild(kvr_ctx *ctx, const kv_weights *weights, const int32_t *token_prefixes,
               const int32_t *prefix_lens, const int32_t *block_tables, int32_t n_requests,
               int32_t max_blocks_per_req, void *stream);

/* Paper Sec. 4.2 (future work: reuse of pool contents instead of a full refill, which needs the
 * caller to track which rows are still consistent): a caller that has verified the first
 * valid_lens[r] rows of request r in the arena (for example a shared prompt whose other
 * sharers are alive) rebuilds only the tail.  Same as kv_rebuild except that tokens
 * [0, valid_lens[r]) are neither recomputed nor written -- their rows stay byte-identical --
 * and the tail attends to them through the block table as it finds them.  valid_lens is a
 * host int32 [n_requests] with 0 <= valid_lens[r] <= prefix_lens[r] (else
 * KVR_ERR_INVALID_ARG); NULL means all zeros, i.e. kv_rebuild. */
int kv_rebuild_from(kvr_ctx *ctx, const kv_weights *weights, const int32_t *token_prefixes,
                    const int32_t *prefix_lens, const int32_t *valid_lens, const int32_t *block_tables,
                    int32_t n_requests, int32_t max_blocks_per_req, void *stream);

/* Checking aid: gather one request's rows of one layer out of the arena into
 * dense [n_tokens, n_kv_heads, head_dim] arrays of the arena's element type.
 * kv_readback copies to host memory and waits for the copy; the _dev variant
 * writes device memory and only enqueues.  Uses the bound workspace as
 * staging (n_tokens * n_kv_heads * head_dim * 2 elements must fit). */
int kv_readback(kvr_ctx *ctx, int32_t layer, const int32_t *block_table_host, int32_t n_tokens,
                void *k_out_host, void *v_out_host, void *stream);
int kv_readback_dev(kvr_ctx *ctx, int32_t layer, const int32_t *block_table_host, int32_t n_tokens,
                    void *k_out_dev, void *v_out_dev, void *stream);

/* No counterpart in the paper: an allocation-free read-back, added for callers
 * that are not in a position to allocate.  Typical cases: a health or
 * consistency probe that runs right after a worker failure, when the device is
 * already filled by the retained weights and KV pool and a cudaMalloc could
 * fail or stall; a standby process that is required to keep its memory
 * footprint fixed; code running under an allocator it does not own.  Such a
 * caller cannot create a context or bind a workspace (both allocate), so this
 * call takes the arena pointer and geometry directly and stages through a
 * fixed array that is part of the library's device image.
 *
 * Same result as kv_readback: the n_tokens rows of one request in one layer,
 * dense [n_tokens, n_kv_heads, head_dim] in the arena's element type, copied to
 * host memory; the call returns after the copies have finished.
 *
 * Limits and rules
 *   - At most KVR_NOALLOC_MAX_BLOCKS table entries and KVR_NOALLOC_MAX_PLANE_BYTES
 *     bytes of K (and the same of V) per call; larger requests return
 *     KVR_ERR_WORKSPACE and do nothing (read a long request in several calls).
 *   - The staging array (16 KiB + 2 x 2 MiB) is held by every GPU that loads
 *     the library until the process exits.
 *   - The first call on a device looks up the array's device address
 *     (cudaGetSymbolAddress).  Every call copies from pageable host memory and
 *     waits for the stream before it returns, so no call, first or later, may be
 *     issued while `stream` is being captured.
 *   - The layer's K and V planes must lie inside the device allocation that
 *     holds arena_dev (its extent is queried from the driver); a geometry that
 *     reaches past it returns KVR_ERR_INVALID_ARG and reads nothing.
 *   - All calls share the one array and it keeps the previous call's bytes;
 *     nothing in it has to start at zero because every byte read back is
 *     written first.  Two calls that overlap in time on one GPU (different
 *     streams or threads) race on it: run them one after the other.
 *   - No cudaMalloc, cudaFree, cudaHostAlloc or other allocating routine is
 *     called; host buffers may be ordinary pageable memory. */
#define KVR_NOALLOC_MAX_BLOCKS 4096
#define KVR_NOALLOC_MAX_PLANE_BYTES (2u << 20)
int kv_readback_noalloc(const void *arena_dev, const kv_arena_geometry *geom, int32_t layer,
                        const int32_t *block_table_host, int32_t n_tokens, void *k_out_host, void *v_out_host,
                        void *stream);

/* Paper Sec. 4.2 step 5 / Sec. 4.3: a recovered request "resumes" generation, i.e. the worker
 * needs the next-token logits after the logged prefix.  With the option "keep_last_hidden" set
 * to 1 before kv_rebuild, the rebuild also keeps the residual-stream row of every request's
 * final token as it enters the last layer (the final token is then always computed, even when
 * its block is shared).  kv_resume_logits finishes the last layer for those R rows only
 * (q projection + RoPE, attention over the request's arena K/V, output projection, SwiGLU
 * MLP), applies the final RMSNorm with `final_gain_dev` [d_model] and multiplies by
 * `lm_head_dev` [vocab, d_model] (both in the model's dtype, 16-byte aligned):
 *     logits_out_dev[r, :] (fp32, [R, vocab])   for the R requests of that rebuild, in order.
 * Every request of the rebuild must have had a non-empty prefix.  Enqueues on `stream`;
 * KVR_ERR_NOT_BOUND if no such rebuild came before.  The kept rows are only read: the call
 * can be repeated after one rebuild and gives the same logits each time. */
int kv_resume_logits(kvr_ctx *ctx, const void *final_gain_dev, const void *lm_head_dev, float *logits_out_dev,
                     void *stream);

/* Paper Sec. 4.2, handover step 2 (pool flush: the old contents are invalidated before any
 * request is rebuilt): overwrite every byte of the bound arena with the 32-bit word `fill_word` (0 for
 * zeros; any NaN pattern to make stale reads visible).  Enqueues on `stream`; HBM-bound. */
int kv_arena_flush(kvr_ctx *ctx, uint32_t fill_word, void *stream);

/* Paper Sec. 4.2, handover step 2 (GPU health check by a small device operation): one small
 * kernel per call, one 64-thread block per SM; every block runs a fixed xorshift32-plus-increment
 * chain (ALU), sums it through shared memory, publishes the result and a flag to global memory
 * and waits -- for at most timeout_ms, never longer -- until it sees its neighbour block's
 * flag (cross-SM visibility).  The flag word is a per-context call counter, so flags left by an
 * earlier call (same seed or not) never satisfy a later call's wait.  The host waits for the
 * kernel for at most 2 x timeout_ms.
 *   KVR_OK                   every block finished, every wait was met, *checksum_out (if not
 *                            NULL) = XOR over blocks b of rotl(result_b, b % 32)
 *   KVR_ERR_DEVICE_TIMEOUT   a device wait ran out or the kernel did not finish in time
 *   KVR_ERR_CUDA             launch or copy failed
 * `seed` selects the chain's start values (result_b is a pure function of seed, b and the
 * thread index), so the caller can check the answer independently. */
int kv_health_probe(kvr_ctx *ctx, uint32_t seed, int32_t timeout_ms, uint32_t *checksum_out, void *stream);

/* Wait for `stream`, then return the device status word (KVR_OK, or
 * KVR_ERR_DEVICE_TIMEOUT if a bounded wait inside a kernel gave up, or
 * KVR_ERR_CUDA if the stream reports an error). */
int kv_sync_status(kvr_ctx *ctx, void *stream);

/* Host-only view of the plan kv_rebuild_from makes for a batch (needs no GPU and no context;
 * inputs are assumed valid, see kv_check_inputs): per request the number of leading tokens that
 * are not computed -- full leading blocks an earlier request of the batch fills completely, rows
 * vouched for by valid_lens (may be NULL), but never the final token when keep_last_hidden is
 * set -- and the totals that follow: computed tokens, chunks of at most chunk_tokens tokens, and
 * attention tiles of at most tile_rows query rows (a tile never spans two requests or chunks).
 * Output pointers may be NULL. */
int kv_plan_host(const int32_t *prefix_lens, const int32_t *valid_lens, const int32_t *block_tables,
                 int32_t n_requests, int32_t max_blocks_per_req, int32_t block_size, int32_t keep_last_hidden,
                 int64_t chunk_tokens, int32_t tile_rows, int32_t *skip_out, int64_t *computed_out,
                 int64_t *chunks_out, int64_t *tiles_out);

/* Host-only validation of a rebuild's inputs against a geometry; needs no GPU
 * and no context.  Same checks, same order and same codes as kv_rebuild. */
int kv_check_inputs(const int32_t *token_prefixes, const int32_t *prefix_lens,
                    const int32_t *block_tables, int32_t n_requests, int32_t max_blocks_per_req,
                    int32_t block_size, int32_t num_blocks, int32_t vocab);

/* Test hooks.  kv_debug_slot_map: slot (block * block_size + offset) of every
 * token of the last kv_rebuild in input order; -1 entries never occur.
 * kv_debug_plan: tokens the last rebuild actually computed (after shared-prefix
 * dedupe), its chunk count and its kernel-launch count. */
int kv_debug_slot_map(kvr_ctx *ctx, int64_t *slots_out_host, int64_t n);
int kv_debug_plan(kvr_ctx *ctx, int64_t *computed_tokens, int64_t *n_chunks, int64_t *n_launches);

/* Per-kernel timing of the last kv_rebuild, for roofline accounting.  With the
 * "profile" option on, kv_rebuild brackets every kernel launch with CUDA events
 * on the caller's stream; this call waits for them and adds up, per kernel
 * kind, the elapsed milliseconds and the number of launches.  Kinds, in order:
 * 0 RoPE table, 1 embedding+RMSNorm, 2 RMSNorm, 3 QKV GEMM (+RoPE+store),
 * 4 attention, 5 output-projection GEMM, 6 gate/up GEMM (+SwiGLU), 7 down GEMM.
 * Arrays hold KVR_N_KINDS entries. */
#define KVR_N_KINDS 8
int kv_debug_profile(kvr_ctx *ctx, double *ms_by_kind, int64_t *launches_by_kind);

/* Options: "keep_last_hidden" 0/1 (see kv_resume_logits; default 0); "probe_mute" 0/1 (test hook: probe blocks do not publish their flags, so every
 * device wait of kv_health_probe runs out; default 0); "wait_limit_ms" 0..60000 (how long a wait inside the tensor-core GEMM and attention
 * kernels may last before the kernel gives up, records KVR_ERR_DEVICE_TIMEOUT for kv_sync_status and returns; 0 = the default of about 2 s);
 * "mute_loads" 0/1 (test hook: the TMA producers of those kernels issue no loads, so every wait on their data runs out and nothing is
 * written; default 0); "profile" 0/1 (see kv_debug_profile; default 0); "gemm" 0 = plain-FMA kernels,
 * 1 = tcgen05 kernels on 128 x 256 tiles, 2 = tcgen05 kernels on CTA pairs (256 x 256 tiles); 1 and 2 are bf16 only, 2 is the default in bf16;
 * "attn" 0 = plain kernel, 1 = warp-level MMA kernel, 2 = tcgen05 kernel (1 and 2 bf16 only; 2 is the
 * default in bf16 and needs block_size 16, otherwise 1 is used); "resume_gemm" 0/1 (kv_resume_logits with the tcgen05
 * kernels and at most 128 requests: 1 = projections by the weight-streaming kernel that cuts the grid along the weight rows
 * and K, the default; 0 = by the rebuild's GEMM); "resume_overlap" 0/1 (on that path, launch every kernel after the first norm
 * so that it may be scheduled while the kernel before it drains; it still waits for that kernel's results; default 1).
 * Returns KVR_ERR_INVALID_ARG for unknown names or values. */
int kv_set_option(kvr_ctx *ctx, const char *name, int64_t value);

/* Standalone access to the GEMM used inside the rebuild, for parity tests:
 * C[M,N] (fp32, dev) = A[M,K] (bf16, dev, row-major) x W[N,K]^T (bf16, dev).
 * impl as in the "gemm" option.  Enqueues on `stream`. */
int kv_debug_gemm(kvr_ctx *ctx, int32_t impl, const void *a_dev, const void *w_dev, float *c_dev,
                  int32_t M, int32_t N, int32_t K, void *stream);

const char *kv_status_str(int status);

#ifdef __cplusplus
}
#endif
#endif /* KVREBUILD_H */
