// C-ABI entry points, host-side validation and planning, and the per-chunk,
// per-layer launch sequence of the rebuild.
#include "kvr_internal.h"

#include <algorithm>
#include <chrono>
#include <cmath>
#include <thread>
#include <cstring>
#include <new>
#include <unordered_map>

using namespace kvr;

namespace {

constexpr size_t ALIGN = 256;
inline size_t align_up(size_t x) { return (x + ALIGN - 1) / ALIGN * ALIGN; }

struct WsLayout {
    size_t h, a, q, m, cs, meta, tables, tiles, part, total;
    size_t l_h, l_h2, l_sk, l_a, l_q, l_m, l_cs, l_pos, l_pairs, l_tiles, l_part;   // per-request buffers for kv_resume_logits
    size_t m_bytes;
};

struct Chunk {
    int64_t off;   // offset into the computed-token stream
    int32_t n;     // tokens
    int32_t tile_begin, tile_end;  // range in the call's attention-tile list
};

}  // namespace

struct kvr_ctx {
    int device = 0;
    int n_sms = 0;
    int *d_status = nullptr;       // device status block: [0] status, [1] flags, [2..3] wait limit in cycles
    int wait_limit_ms = 0;         // 0 = the default of about two seconds
    int mute_loads = 0;
    // arena
    bool arena_bound = false;
    kv_arena_geometry geom{};
    ArenaView av{};
    // weights
    bool weights_bound = false;
    kv_model_desc desc{};
    ModelDims md{};
    const void *embed = nullptr;
    std::vector<const void *> w[9];  // ln1 wq wk wv wo ln2 wg wu wd
    std::vector<CUtensorMap> tm_w[9];
    std::vector<const void *> vx[5];  // optional bq bk bv qn kn (empty = absent)
    bool tc_ready = false;
    // workspace
    bool ws_bound = false;
    char *ws = nullptr;
    size_t ws_bytes = 0;
    int64_t max_chunk = 0;
    int32_t max_req = 0, max_blk = 0;
    WsLayout lay{};
    CUtensorMap tm_a_d{}, tm_a_q{}, tm_m{}, tm_q{}, tm_kv{}, tm_h{};
    bool tm_kv_ok = false;
    // pinned staging
    char *pinned = nullptr;
    size_t pinned_bytes = 0;
    cudaEvent_t staging_free = nullptr;
    bool staging_busy = false;
    // tensor-parallel rank (tp_world 1 = unsharded)
    int tp_world = 1, tp_rank = 0;
    kv_allreduce_fn tp_allreduce = nullptr;
    void *tp_user = nullptr;
    // options
    int gemm_impl = 2, attn_impl = 2, profile = 0, probe_mute = 0;
    int resume_pdl = 1;
    int resume_gemm = 1;           // kv_resume_logits: 1 = weight-streaming GEMM for up to 128 requests, 0 = the rebuild's GEMM
    uint32_t *d_probe = nullptr;   // [2 * PROBE_MAX_BLOCKS]: flags, results
    uint32_t probe_epoch = 0;      // word the current probe publishes; never 0, never reused by the next call
    int clock_khz = 0;
    // per-launch event pairs of the last call (profile mode)
    std::vector<cudaEvent_t> ev_pool;
    std::vector<int> ev_kind;   // kind of pair i (events 2i, 2i+1)
    // last-call records
    std::vector<int64_t> last_slots;
    int64_t last_computed = 0, last_chunks = 0, last_launches = 0;
    // resume logits: residual rows of every request's final token, kept by the last rebuild
    int keep_last = 0;
    bool have_last = false;
    bool dev_tables_current = false;   // the workspace still holds the last rebuild's block tables
    std::vector<int32_t> last_lens, last_tables;
    int32_t last_width = 0;
    CUtensorMap tm_la_d{}, tm_la_q{}, tm_lm{}, tm_lq{}, tm_lh{};
    CUtensorMap tm_x_d{}, tm_x_q{}, tm_x_m{};   // l_a and l_m again, box of x_rows rows (weight-streaming GEMM)
    int x_rows = 128;
};

namespace {

enum { W_LN1 = 0, W_WQ, W_WK, W_WV, W_WO, W_LN2, W_WG, W_WU, W_WD };

// Flags and wait limit of the device status block (the status word itself is left alone).
static int write_status_block(kvr_ctx *c) {
    const long long ms = c->wait_limit_ms > 0 ? c->wait_limit_ms : 2000;
    int32_t words[3];
    const long long cycles = ms * (long long)std::max(c->clock_khz, 1000);
    words[0] = c->mute_loads ? 1 : 0;
    std::memcpy(&words[1], &cycles, sizeof(cycles));
    return cudaMemcpy(c->d_status + 1, words, sizeof(words), cudaMemcpyHostToDevice) == cudaSuccess ? KVR_OK
                                                                                                     : KVR_ERR_CUDA;
}

// optional projection terms of layer l (null pointers where the bound set has none)
static QkvExtras qkv_extras(const kvr_ctx *c, int l) {
    QkvExtras ex;
    if (!c->vx[0].empty()) { ex.bq = c->vx[0][l]; ex.bk = c->vx[1][l]; ex.bv = c->vx[2][l]; }
    if (!c->vx[3].empty()) { ex.qn = c->vx[3][l]; ex.kn = c->vx[4][l]; }
    ex.eps = c->md.eps;
    return ex;
}
static void set_tc_extras(TcGemmEpilogue &ep, const QkvExtras &ex, bool with_q) {
    ep.bias_q = with_q ? (const __nv_bfloat16 *)ex.bq : nullptr;
    ep.bias_k = (const __nv_bfloat16 *)ex.bk;
    ep.bias_v = (const __nv_bfloat16 *)ex.bv;
    ep.gain_q = with_q ? (const __nv_bfloat16 *)ex.qn : nullptr;
    ep.gain_k = (const __nv_bfloat16 *)ex.kn;
    ep.qk_eps = ex.eps;
}

inline bool is_fp32(const kvr_ctx *c) { return c->desc.dtype == KVR_FP32; }
inline size_t esize(int dtype) { return dtype == KVR_FP32 ? 4 : 2; }

bool compute_layout(const kvr_ctx *c, int64_t Tc, int32_t max_req, int32_t max_blk, WsLayout *L) {
    if (!c->weights_bound || Tc <= 0 || max_req <= 0 || max_blk <= 0) return false;
    const ModelDims &md = c->md;
    const size_t es = esize(c->desc.dtype);
    const size_t T = (size_t)Tc;
    size_t o = 0;
    L->h = o; o += align_up(T * md.d * sizeof(float));
    L->a = o; o += align_up(T * (size_t)std::max(md.d, md.q_dim) * es);
    L->q = o; o += align_up(T * (size_t)md.q_dim * es);
    L->m_bytes = std::max(T * (size_t)md.F * es, T * (size_t)(md.q_dim + 2 * md.kv_dim) * sizeof(float));
    L->m = o; o += align_up(L->m_bytes);
    L->cs = o; o += align_up(T * (size_t)(md.hd / 2) * sizeof(float2));
    L->meta = o; o += align_up(T * 4 * sizeof(int32_t));
    L->tables = o; o += align_up((size_t)max_req * max_blk * sizeof(int32_t));
    const size_t max_tiles = T / ATTN_TILE_Q + (size_t)max_req + 1;
    L->tiles = o; o += align_up(max_tiles * sizeof(AttnTile));
    const size_t Rq = (size_t)max_req;
    L->l_h = o; o += align_up(Rq * md.d * sizeof(float));    // kept by the rebuild, read-only for the resume call
    L->l_h2 = o; o += align_up(Rq * md.d * sizeof(float));   // the resume call's own residual rows
    L->l_sk = o;   // partial products of the K splits of the weight-streaming GEMM
    o += align_up((size_t)GEMM_SKINNY_MAX_SPLITS * Rq * (size_t)std::max(md.d, md.q_dim) * sizeof(float));
    L->l_a = o; o += align_up(Rq * (size_t)std::max(md.d, md.q_dim) * es);
    L->l_q = o; o += align_up(Rq * (size_t)md.q_dim * es);
    L->l_m = o; o += align_up(std::max(Rq * (size_t)md.F * es, Rq * (size_t)md.q_dim * sizeof(float)));
    L->l_cs = o; o += align_up(Rq * (size_t)(md.hd / 2) * sizeof(float2));
    L->l_pos = o; o += align_up(Rq * 2 * sizeof(int32_t));
    L->l_pairs = o; o += align_up(Rq * sizeof(int2));
    L->l_tiles = o; o += align_up(Rq * sizeof(AttnTile));
    L->l_part = o; o += align_up(attn_decode_scratch_bytes(max_req, md.Hq, md.hd));
    L->part = o;
    if (c->tp_world > 1) o += align_up(T * md.d * sizeof(float));   // partial sums awaiting the all-reduce
    L->total = o;
    return true;
}

int validate_inputs(const int32_t *tokens, const int32_t *lens, const int32_t *tables, int32_t R, int32_t width,
                    int32_t B, int32_t NB, int32_t V) {
    if (R < 0 || width < 0 || B <= 0 || NB <= 0 || V <= 0) return KVR_ERR_INVALID_ARG;
    if (R == 0) return KVR_OK;
    if (!lens) return KVR_ERR_INVALID_ARG;
    int64_t total = 0;
    for (int r = 0; r < R; ++r) {
        if (lens[r] < 0) return KVR_ERR_INVALID_ARG;
        total += lens[r];
    }
    if (total > 0 && (!tokens || !tables)) return KVR_ERR_INVALID_ARG;
    for (int r = 0; r < R; ++r) {
        const int need = (lens[r] + B - 1) / B;
        if (need > width) return KVR_ERR_TABLE_TOO_SHORT;
        for (int j = 0; j < need; ++j)
            if (tables[(int64_t)r * width + j] == -1) return KVR_ERR_TABLE_TOO_SHORT;
    }
    for (int r = 0; r < R; ++r) {
        const int need = (lens[r] + B - 1) / B;
        for (int j = 0; j < need; ++j) {
            const int32_t b = tables[(int64_t)r * width + j];
            if (b < 0 || b >= NB) return KVR_ERR_BLOCK_OOB;
        }
    }
    for (int64_t i = 0; i < total; ++i)
        if (tokens[i] < 0 || tokens[i] >= V) return KVR_ERR_TOKEN_OOB;
    // aliasing
    std::vector<int64_t> start(R + 1, 0);
    for (int r = 0; r < R; ++r) start[r + 1] = start[r] + lens[r];
    struct Own { int r, j; };
    std::unordered_map<int32_t, Own> owner;
    owner.reserve((size_t)(total / B + R) * 2 + 16);
    for (int r = 0; r < R; ++r) {
        const int need = (lens[r] + B - 1) / B;
        int prev_owner = -1;  // owner request of block j-1 if it was a verified share
        for (int j = 0; j < need; ++j) {
            const int32_t b = tables[(int64_t)r * width + j];
            auto it = owner.find(b);
            if (it == owner.end()) {
                owner.emplace(b, Own{r, j});
                prev_owner = -1;
                continue;
            }
            const Own o = it->second;
            if (o.r == r || o.j != j) return KVR_ERR_ALIAS_CONFLICT;
            const int64_t common = std::min<int64_t>(std::min(lens[r], lens[o.r]), (int64_t)(j + 1) * B);
            // if block j-1 was shared with the same request, tokens [0, jB) already matched
            const int64_t from = (prev_owner == o.r) ? (int64_t)j * B : 0;
            if (common > from &&
                std::memcmp(tokens + start[r] + from, tokens + start[o.r] + from,
                            (size_t)(common - from) * sizeof(int32_t)) != 0)
                return KVR_ERR_ALIAS_CONFLICT;
            prev_owner = o.r;
            if (lens[r] > lens[o.r]) it->second = Own{r, j};
        }
    }
    return KVR_OK;
}

#define CU_OK(x)                                  \
    do {                                          \
        if ((x) != cudaSuccess) return KVR_ERR_CUDA; \
    } while (0)

struct SetDevice {
    int prev = -1;
    bool ok = true;
    explicit SetDevice(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    }
    ~SetDevice() { if (prev >= 0) cudaSetDevice(prev); }
};

// Per-request metadata of kv_resume_logits: [pos R][table row R] and one single-row attention tile per request
// (longest context first).  Written by the rebuild that keeps the final rows, so the resume call copies nothing.
static size_t resume_meta_bytes(int R) {
    return align_up((size_t)R * 2 * sizeof(int32_t)) + align_up((size_t)R * sizeof(AttnTile));
}
static int upload_resume_meta(kvr_ctx *c, char *staging, const int32_t *lens, int R, cudaStream_t s) {
    int32_t *st_pos = (int32_t *)staging;
    AttnTile *st_tiles = (AttnTile *)(staging + align_up((size_t)R * 2 * sizeof(int32_t)));
    for (int r = 0; r < R; ++r) {
        st_pos[r] = lens[r] - 1;
        st_pos[R + r] = r;
        st_tiles[r] = AttnTile{r, lens[r] - 1, 1, r};
    }
    std::stable_sort(st_tiles, st_tiles + R, [](const AttnTile &x, const AttnTile &y) { return x.pos0 > y.pos0; });
    CU_OK(cudaMemcpyAsync(c->ws + c->lay.l_pos, st_pos, (size_t)R * 2 * sizeof(int32_t), cudaMemcpyHostToDevice, s));
    CU_OK(cudaMemcpyAsync(c->ws + c->lay.l_tiles, st_tiles, (size_t)R * sizeof(AttnTile), cudaMemcpyHostToDevice, s));
    return KVR_OK;
}

int ensure_staging(kvr_ctx *c, size_t bytes) {
    if (c->staging_busy) {
        CU_OK(cudaEventSynchronize(c->staging_free));
        c->staging_busy = false;
    }
    if (bytes <= c->pinned_bytes) return KVR_OK;
    if (c->pinned) cudaFreeHost(c->pinned);
    c->pinned = nullptr;
    c->pinned_bytes = 0;
    const size_t want = std::max(bytes, (size_t)1 << 16);
    CU_OK(cudaHostAlloc((void **)&c->pinned, want, cudaHostAllocDefault));
    c->pinned_bytes = want;
    return KVR_OK;
}

// Brackets one launch with events when profiling is on.
struct Timed {
    kvr_ctx *c;
    cudaStream_t s;
    bool on;
    Timed(kvr_ctx *c_, int kind, cudaStream_t s_) : c(c_), s(s_), on(c_->profile != 0) {
        if (!on) return;
        const size_t i = c->ev_kind.size();
        while (c->ev_pool.size() < 2 * (i + 1)) {
            cudaEvent_t e;
            if (cudaEventCreate(&e) != cudaSuccess) { on = false; return; }
            c->ev_pool.push_back(e);
        }
        c->ev_kind.push_back(kind);
        cudaEventRecord(c->ev_pool[2 * i], s);
    }
    ~Timed() {
        if (on) cudaEventRecord(c->ev_pool[2 * (c->ev_kind.size() - 1) + 1], s);
    }
};

// Which leading tokens of each request are not computed: full leading blocks that an earlier
// request of the batch fills completely (shared prefixes are computed once), rows the caller
// vouches for (valid_lens, may be null), but never the final token when its hidden state is kept.
void plan_skips(const int32_t *lens, const int32_t *tables, const int32_t *valid_lens, int R, int width, int B,
                bool keep_last, std::vector<int32_t> &skip) {
    skip.assign((size_t)R, 0);
    int64_t total = 0;
    for (int r = 0; r < R; ++r) total += lens[r];
    std::unordered_map<int32_t, char> full;  // blocks some earlier request fills completely
    full.reserve((size_t)(total / B + R) * 2 + 16);
    for (int r = 0; r < R; ++r) {
        const int need = (lens[r] + B - 1) / B;
        int lead = 0;
        while (lead < need && full.count(tables[(int64_t)r * width + lead])) ++lead;
        skip[r] = (int32_t)std::min<int64_t>(lens[r], (int64_t)lead * B);
        if (valid_lens) skip[r] = std::max(skip[r], valid_lens[r]);
        if (keep_last && lens[r] > 0) skip[r] = std::min<int32_t>(skip[r], lens[r] - 1);
        for (int j = 0; j < lens[r] / B; ++j) full.emplace(tables[(int64_t)r * width + j], 1);
    }
}

}  // namespace

extern "C" {

const char *kv_status_str(int s) {
    switch (s) {
        case KVR_OK: return "KVR_OK";
        case KVR_ERR_INVALID_ARG: return "KVR_ERR_INVALID_ARG";
        case KVR_ERR_NOT_BOUND: return "KVR_ERR_NOT_BOUND";
        case KVR_ERR_UNSUPPORTED: return "KVR_ERR_UNSUPPORTED";
        case KVR_ERR_BLOCK_OOB: return "KVR_ERR_BLOCK_OOB";
        case KVR_ERR_TABLE_TOO_SHORT: return "KVR_ERR_TABLE_TOO_SHORT";
        case KVR_ERR_ALIAS_CONFLICT: return "KVR_ERR_ALIAS_CONFLICT";
        case KVR_ERR_TOKEN_OOB: return "KVR_ERR_TOKEN_OOB";
        case KVR_ERR_WORKSPACE: return "KVR_ERR_WORKSPACE";
        case KVR_ERR_CUDA: return "KVR_ERR_CUDA";
        case KVR_ERR_DEVICE_TIMEOUT: return "KVR_ERR_DEVICE_TIMEOUT";
        default: return "KVR_ERR_UNKNOWN";
    }
}

int kv_check_inputs(const int32_t *tokens, const int32_t *lens, const int32_t *tables, int32_t R, int32_t width,
                    int32_t block_size, int32_t num_blocks, int32_t vocab) {
    return validate_inputs(tokens, lens, tables, R, width, block_size, num_blocks, vocab);
}

int kv_plan_host(const int32_t *lens, const int32_t *valid_lens, const int32_t *tables, int32_t R, int32_t width,
                 int32_t block_size, int32_t keep_last_hidden, int64_t chunk_tokens, int32_t tile_rows,
                 int32_t *skip_out, int64_t *computed_out, int64_t *chunks_out, int64_t *tiles_out) {
    if (R < 0 || width < 0 || block_size <= 0 || chunk_tokens <= 0 || tile_rows <= 0) return KVR_ERR_INVALID_ARG;
    if (R > 0 && (!lens || !tables)) return KVR_ERR_INVALID_ARG;
    for (int r = 0; r < R; ++r) {
        if (lens[r] < 0 || (int64_t)(lens[r] + block_size - 1) / block_size > width) return KVR_ERR_INVALID_ARG;
        if (valid_lens && (valid_lens[r] < 0 || valid_lens[r] > lens[r])) return KVR_ERR_INVALID_ARG;
    }
    std::vector<int32_t> skip;
    plan_skips(lens, tables, valid_lens, R, width, block_size, keep_last_hidden != 0, skip);
    // the computed stream is cut into chunks at token granularity; a request's run inside a chunk
    // is cut into attention tiles of at most tile_rows query rows
    int64_t T = 0, tiles = 0, g = 0;
    for (int r = 0; r < R; ++r) {
        T += lens[r] - skip[r];
        int64_t left = lens[r] - skip[r];
        while (left > 0) {
            const int64_t room = chunk_tokens - g % chunk_tokens;
            const int64_t run = std::min(left, room);
            tiles += (run + tile_rows - 1) / tile_rows;
            g += run;
            left -= run;
        }
        if (skip_out) skip_out[r] = skip[r];
    }
    if (computed_out) *computed_out = T;
    if (chunks_out) *chunks_out = (T + chunk_tokens - 1) / chunk_tokens;
    if (tiles_out) *tiles_out = tiles;
    return KVR_OK;
}

int kv_ctx_create(kvr_ctx **out, int device) {
    if (!out) return KVR_ERR_INVALID_ARG;
    *out = nullptr;
    int n = 0;
    if (cudaGetDeviceCount(&n) != cudaSuccess || device < 0 || device >= n) return KVR_ERR_CUDA;
    SetDevice sd(device);
    if (!sd.ok) return KVR_ERR_CUDA;
    kvr_ctx *c = new (std::nothrow) kvr_ctx();
    if (!c) return KVR_ERR_INVALID_ARG;
    c->device = device;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) { delete c; return KVR_ERR_CUDA; }
    c->n_sms = prop.multiProcessorCount;
    cudaDeviceGetAttribute(&c->clock_khz, cudaDevAttrClockRate, device);
    if (cudaMalloc((void **)&c->d_status, 4 * sizeof(int)) != cudaSuccess ||
        cudaMalloc((void **)&c->d_probe, 2 * PROBE_MAX_BLOCKS * sizeof(uint32_t)) != cudaSuccess ||
        cudaMemset(c->d_probe, 0, 2 * PROBE_MAX_BLOCKS * sizeof(uint32_t)) != cudaSuccess ||
        cudaMemset(c->d_status, 0, 4 * sizeof(int)) != cudaSuccess || write_status_block(c) != KVR_OK ||
        cudaEventCreateWithFlags(&c->staging_free, cudaEventDisableTiming) != cudaSuccess) {
        delete c;
        return KVR_ERR_CUDA;
    }
    c->tc_ready = (prop.major == 10) && tc_gemm_init(device) == KVR_OK && attn_tc_init(device) == KVR_OK &&
                  attn_fa_init(device) == KVR_OK && gemm_skinny_init(device) == KVR_OK;
    *out = c;
    return KVR_OK;
}

int kv_ctx_destroy(kvr_ctx *c) {
    if (!c) return KVR_ERR_INVALID_ARG;
    SetDevice sd(c->device);
    if (c->staging_busy) cudaEventSynchronize(c->staging_free);
    if (c->pinned) cudaFreeHost(c->pinned);
    for (cudaEvent_t e : c->ev_pool) cudaEventDestroy(e);
    if (c->d_status) cudaFree(c->d_status);
    if (c->d_probe) cudaFree(c->d_probe);
    if (c->staging_free) cudaEventDestroy(c->staging_free);
    delete c;
    return KVR_OK;
}

int kv_arena_bind(kvr_ctx *c, void *arena, size_t bytes, const kv_arena_geometry *g) {
    if (!c || !arena || !g) return KVR_ERR_INVALID_ARG;
    if (g->block_size <= 0 || g->num_blocks <= 0 || g->n_layers <= 0 || g->n_kv_heads <= 0 || g->head_dim <= 0 ||
        (g->dtype != KVR_BF16 && g->dtype != KVR_FP32))
        return KVR_ERR_INVALID_ARG;
    if (((uintptr_t)arena) % ALIGN) return KVR_ERR_INVALID_ARG;
    const int64_t row = (int64_t)g->n_kv_heads * g->head_dim;
    const int64_t slots = (int64_t)g->num_blocks * g->block_size;
    if (slots >= ((int64_t)1 << 31)) return KVR_ERR_UNSUPPORTED;
    const size_t need = (size_t)g->n_layers * 2 * (size_t)slots * (size_t)row * esize(g->dtype);
    if (bytes < need) return KVR_ERR_INVALID_ARG;
    if ((row * esize(g->dtype)) % 16) return KVR_ERR_UNSUPPORTED;
    if (c->weights_bound) {
        const kv_model_desc &d = c->desc;
        if (d.n_layers != g->n_layers || d.n_kv_heads != g->n_kv_heads || d.head_dim != g->head_dim ||
            d.dtype != g->dtype)
            return KVR_ERR_INVALID_ARG;
    }
    c->geom = *g;
    c->av.base = arena;
    c->av.row = (int32_t)row;
    c->av.kv_stride = slots * row;
    c->av.layer_stride = 2 * slots * row;
    c->av.block_size = g->block_size;
    c->av.num_blocks = g->num_blocks;
    c->av.n_kv_heads = g->n_kv_heads;
    c->av.head_dim = g->head_dim;
    c->tm_kv_ok = false;
    if (g->dtype == KVR_BF16 && c->tc_ready && g->block_size == 16 && (row % 64) == 0 &&
        (g->head_dim == 64 || g->head_dim == 128)) {
        const int64_t rows2d = (int64_t)g->n_layers * 2 * slots;
        if (rows2d < ((int64_t)1 << 31) &&
            tc_make_tmap_kv(&c->tm_kv, arena, rows2d, row, g->head_dim / 64) == KVR_OK)
            c->tm_kv_ok = true;
    }
    c->arena_bound = true;
    return KVR_OK;
}

int kv_weights_bind(kvr_ctx *c, const kv_model_desc *d, const kv_weights *w) {
    if (!c || !d || !w) return KVR_ERR_INVALID_ARG;
    if (d->n_layers <= 0 || d->d_model <= 0 || d->n_q_heads <= 0 || d->n_kv_heads <= 0 || d->head_dim <= 0 ||
        d->ffn <= 0 || d->vocab <= 0 || !(d->rms_eps >= 0.f) || !(d->rope_base > 0.f) ||
        (d->dtype != KVR_BF16 && d->dtype != KVR_FP32))
        return KVR_ERR_INVALID_ARG;
    if (d->n_q_heads % d->n_kv_heads) return KVR_ERR_INVALID_ARG;
    if (d->head_dim != 64 && d->head_dim != 128) return KVR_ERR_UNSUPPORTED;
    if (d->d_model % 8 || d->ffn % 8) return KVR_ERR_UNSUPPORTED;
    const void *const *src[9] = {w->ln1, w->wq, w->wk, w->wv, w->wo, w->ln2, w->wg, w->wu, w->wd};
    if (!w->embed) return KVR_ERR_INVALID_ARG;
    for (int k = 0; k < 9; ++k) {
        if (!src[k]) return KVR_ERR_INVALID_ARG;
        for (int l = 0; l < d->n_layers; ++l)
            if (!src[k][l] || ((uintptr_t)src[k][l]) % 16) return KVR_ERR_INVALID_ARG;
    }
    if (c->arena_bound) {
        const kv_arena_geometry &g = c->geom;
        if (d->n_layers != g.n_layers || d->n_kv_heads != g.n_kv_heads || d->head_dim != g.head_dim ||
            d->dtype != g.dtype)
            return KVR_ERR_INVALID_ARG;
    }
    SetDevice sd(c->device);
    c->desc = *d;
    ModelDims &md = c->md;
    md.L = d->n_layers; md.d = d->d_model; md.Hq = d->n_q_heads; md.Hkv = d->n_kv_heads; md.hd = d->head_dim;
    md.F = d->ffn; md.V = d->vocab; md.q_dim = md.Hq * md.hd; md.kv_dim = md.Hkv * md.hd;
    md.eps = d->rms_eps; md.rope_base = (double)d->rope_base;
    c->embed = w->embed;
    for (int k = 0; k < 9; ++k) c->w[k].assign(src[k], src[k] + d->n_layers);
    for (int k = 0; k < 9; ++k) c->tm_w[k].clear();
    for (int k = 0; k < 5; ++k) c->vx[k].clear();
    if (d->dtype == KVR_BF16 && c->tc_ready) {
        const int rows[9] = {0, md.q_dim, md.kv_dim, md.kv_dim, md.d, 0, md.F, md.F, md.d};
        const int cols[9] = {0, md.d, md.d, md.d, md.q_dim, 0, md.d, md.d, md.F};
        for (int k = 0; k < 9; ++k) {
            if (!rows[k]) continue;
            c->tm_w[k].resize(d->n_layers);
            for (int l = 0; l < d->n_layers; ++l) {
                int st = tc_make_tmap_2d(&c->tm_w[k][l], c->w[k][l], rows[k], cols[k], 128, 64);
                if (st != KVR_OK) return st;
            }
        }
    }
    c->weights_bound = true;
    c->ws_bound = false;  // layout depends on the shape
    return KVR_OK;
}

int kv_variant_bind(kvr_ctx *c, const kv_proj_variant *v) {
    if (!c) return KVR_ERR_INVALID_ARG;
    if (!c->weights_bound) return KVR_ERR_NOT_BOUND;
    std::vector<const void *> nv[5];
    if (v) {
        const void *const *src[5] = {v->bq, v->bk, v->bv, v->q_norm, v->k_norm};
        // biases come as a set, norm gains as a pair
        if ((!!src[0] != !!src[1]) || (!!src[0] != !!src[2]) || (!!src[3] != !!src[4])) return KVR_ERR_INVALID_ARG;
        for (int k = 0; k < 5; ++k) {
            if (!src[k]) continue;
            for (int l = 0; l < c->md.L; ++l)
                if (!src[k][l] || ((uintptr_t)src[k][l]) % 16) return KVR_ERR_INVALID_ARG;
            nv[k].assign(src[k], src[k] + c->md.L);
        }
    }
    for (int k = 0; k < 5; ++k) c->vx[k].swap(nv[k]);
    return KVR_OK;
}

int kv_tp_plan_host(const kv_model_desc *full, int32_t tp_world, int32_t tp_rank, kv_model_desc *local_out,
                    kv_tp_shard *shard_out) {
    if (!full || tp_world < 1 || tp_rank < 0 || tp_rank >= tp_world) return KVR_ERR_INVALID_ARG;
    if (full->n_q_heads <= 0 || full->n_kv_heads <= 0 || full->ffn <= 0 || full->n_q_heads % full->n_kv_heads)
        return KVR_ERR_INVALID_ARG;
    if (full->n_kv_heads % tp_world || full->ffn % (8 * tp_world)) return KVR_ERR_UNSUPPORTED;
    const int G = full->n_q_heads / full->n_kv_heads;
    kv_tp_shard sh;
    sh.n_kv_heads = full->n_kv_heads / tp_world;
    sh.kv_head0 = tp_rank * sh.n_kv_heads;
    sh.n_q_heads = sh.n_kv_heads * G;            // whole GQA groups: a rank's q heads read only its kv heads
    sh.q_head0 = sh.kv_head0 * G;
    sh.ffn = full->ffn / tp_world;
    sh.ffn0 = tp_rank * sh.ffn;
    if (shard_out) *shard_out = sh;
    if (local_out) {
        *local_out = *full;
        local_out->n_q_heads = sh.n_q_heads;
        local_out->n_kv_heads = sh.n_kv_heads;
        local_out->ffn = sh.ffn;
    }
    return KVR_OK;
}

int kv_tp_bind(kvr_ctx *c, const kv_tp_config *cfg) {
    if (!c) return KVR_ERR_INVALID_ARG;
    if (!c->weights_bound) return KVR_ERR_NOT_BOUND;
    if (!cfg || cfg->tp_world <= 1) {
        if (cfg && cfg->tp_world < 1) return KVR_ERR_INVALID_ARG;
        c->tp_world = 1; c->tp_rank = 0; c->tp_allreduce = nullptr; c->tp_user = nullptr;
    } else {
        if (cfg->tp_rank < 0 || cfg->tp_rank >= cfg->tp_world || !cfg->allreduce) return KVR_ERR_INVALID_ARG;
        c->tp_world = cfg->tp_world; c->tp_rank = cfg->tp_rank;
        c->tp_allreduce = cfg->allreduce; c->tp_user = cfg->user;
    }
    c->ws_bound = false;   // the layout depends on it
    return KVR_OK;
}

size_t kv_workspace_bytes(const kvr_ctx *c, int64_t max_chunk_tokens, int32_t max_requests,
                          int32_t max_blocks_per_req) {
    WsLayout L;
    if (!c || !compute_layout(c, max_chunk_tokens, max_requests, max_blocks_per_req, &L)) return 0;
    return L.total;
}

int kv_workspace_bind(kvr_ctx *c, void *ws, size_t bytes, int64_t max_chunk_tokens, int32_t max_requests,
                      int32_t max_blocks_per_req) {
    if (!c || !ws) return KVR_ERR_INVALID_ARG;
    if (!c->weights_bound) return KVR_ERR_NOT_BOUND;
    if (((uintptr_t)ws) % ALIGN) return KVR_ERR_INVALID_ARG;
    if (max_chunk_tokens >= ((int64_t)1 << 30)) return KVR_ERR_UNSUPPORTED;
    WsLayout L;
    if (!compute_layout(c, max_chunk_tokens, max_requests, max_blocks_per_req, &L)) return KVR_ERR_INVALID_ARG;
    if (bytes < L.total) return KVR_ERR_WORKSPACE;
    SetDevice sd(c->device);
    c->ws = (char *)ws;
    c->ws_bytes = bytes;
    c->max_chunk = max_chunk_tokens;
    c->max_req = max_requests;
    c->max_blk = max_blocks_per_req;
    c->lay = L;
    if (c->desc.dtype == KVR_BF16 && c->tc_ready) {
        const ModelDims &md = c->md;
        int st = tc_make_tmap_2d(&c->tm_a_d, c->ws + L.a, max_chunk_tokens, md.d, 128, 64);
        if (st == KVR_OK) st = tc_make_tmap_2d(&c->tm_a_q, c->ws + L.a, max_chunk_tokens, md.q_dim, 128, 64);
        if (st == KVR_OK) st = tc_make_tmap_2d(&c->tm_m, c->ws + L.m, max_chunk_tokens, md.F, 128, 64);
        if (st == KVR_OK) st = tc_make_tmap_2d(&c->tm_q, c->ws + L.q, max_chunk_tokens, md.q_dim, 128, 64);
        if (st == KVR_OK) st = tc_make_tmap_f32(&c->tm_h, c->ws + L.h, max_chunk_tokens, md.d);
        if (st == KVR_OK) st = tc_make_tmap_2d(&c->tm_la_d, c->ws + L.l_a, max_requests, md.d, 128, 64);
        if (st == KVR_OK) st = tc_make_tmap_2d(&c->tm_la_q, c->ws + L.l_a, max_requests, md.q_dim, 128, 64);
        if (st == KVR_OK) st = tc_make_tmap_2d(&c->tm_lm, c->ws + L.l_m, max_requests, md.F, 128, 64);
        if (st == KVR_OK) st = tc_make_tmap_2d(&c->tm_lq, c->ws + L.l_q, max_requests, md.q_dim, 128, 64);
        c->x_rows = max_requests <= 64 ? 64 : 128;
        if (st == KVR_OK) st = tc_make_tmap_2d(&c->tm_x_d, c->ws + L.l_a, max_requests, md.d, c->x_rows, 64);
        if (st == KVR_OK) st = tc_make_tmap_2d(&c->tm_x_q, c->ws + L.l_a, max_requests, md.q_dim, c->x_rows, 64);
        if (st == KVR_OK) st = tc_make_tmap_2d(&c->tm_x_m, c->ws + L.l_m, max_requests, md.F, c->x_rows, 64);
        if (st == KVR_OK) st = tc_make_tmap_f32(&c->tm_lh, c->ws + L.l_h2, max_requests, md.d);
        if (st != KVR_OK) return st;
    }
    c->ws_bound = true;
    c->dev_tables_current = false;
    return KVR_OK;
}

int kv_set_option(kvr_ctx *c, const char *name, int64_t value) {
    if (!c || !name) return KVR_ERR_INVALID_ARG;
    if (!std::strcmp(name, "attn")) {
        if (value < 0 || value > 2) return KVR_ERR_INVALID_ARG;
        c->attn_impl = (int)value;
        return KVR_OK;
    }
    if (!std::strcmp(name, "gemm")) {
        if (value < 0 || value > 2) return KVR_ERR_INVALID_ARG;
        c->gemm_impl = (int)value;
        return KVR_OK;
    }
    if (!std::strcmp(name, "resume_gemm")) {
        if (value < 0 || value > 1) return KVR_ERR_INVALID_ARG;
        c->resume_gemm = (int)value;
        return KVR_OK;
    }
    if (!std::strcmp(name, "wait_limit_ms")) {
        if (value < 0 || value > 60000) return KVR_ERR_INVALID_ARG;
        SetDevice sd(c->device);
        c->wait_limit_ms = (int)value;
        return write_status_block(c);
    }
    if (value != 0 && value != 1) return KVR_ERR_INVALID_ARG;
    if (!std::strcmp(name, "mute_loads")) {
        SetDevice sd(c->device);
        c->mute_loads = (int)value;
        return write_status_block(c);
    }
    if (!std::strcmp(name, "profile")) { c->profile = (int)value; return KVR_OK; }
    if (!std::strcmp(name, "resume_overlap")) { c->resume_pdl = (int)value; return KVR_OK; }
    if (!std::strcmp(name, "probe_mute")) { c->probe_mute = (int)value; return KVR_OK; }
    if (!std::strcmp(name, "keep_last_hidden")) { c->keep_last = (int)value; return KVR_OK; }
    return KVR_ERR_INVALID_ARG;
}

int kv_rebuild(kvr_ctx *c, const kv_weights *weights, const int32_t *tokens, const int32_t *lens,
               const int32_t *tables, int32_t R, int32_t width, void *stream_v) {
    return kv_rebuild_from(c, weights, tokens, lens, nullptr, tables, R, width, stream_v);
}

int kv_rebuild_from(kvr_ctx *c, const kv_weights *weights, const int32_t *tokens, const int32_t *lens,
                    const int32_t *valid_lens, const int32_t *tables, int32_t R, int32_t width, void *stream_v) {
    if (!c) return KVR_ERR_INVALID_ARG;
    if (!c->arena_bound || !c->weights_bound || !c->ws_bound) return KVR_ERR_NOT_BOUND;
    if (weights && weights->embed != c->embed) return KVR_ERR_UNSUPPORTED;
    const ModelDims &md = c->md;
    const int B = c->geom.block_size;
    int st = validate_inputs(tokens, lens, tables, R, width, B, c->geom.num_blocks, md.V);
    if (st != KVR_OK) return st;
    if (valid_lens)
        for (int r = 0; r < R; ++r)
            if (valid_lens[r] < 0 || valid_lens[r] > lens[r]) return KVR_ERR_INVALID_ARG;
    if (R > c->max_req || width > c->max_blk) return KVR_ERR_WORKSPACE;
    const bool fp32 = is_fp32(c);
    const bool use_tc_gemm = !fp32 && c->gemm_impl >= 1;
    // The fused QKV epilogue hands every 128-column half tile to exactly one of q, k, v, so it needs
    // q_dim and kv_dim to be multiples of 128; other head counts take the plain projection + RoPE/scatter
    // kernels for this one step (same arena rows, no tile ever straddles two destinations).
    const bool use_tc_qkv = use_tc_gemm && md.q_dim % 128 == 0 && md.kv_dim % 128 == 0;
    // tcgen05 attention needs 16-slot blocks: otherwise the warp-MMA kernel takes over
    const bool use_fa_attn = !fp32 && c->attn_impl >= 2 && c->tm_kv_ok;
    const bool use_tc_attn = !fp32 && (c->attn_impl == 1 || (c->attn_impl >= 2 && !use_fa_attn));
    const int tile_q = use_fa_attn ? ATTN_FA_TILE_Q : ATTN_TILE_Q;
    if ((use_tc_gemm || use_tc_attn || use_fa_attn) && !c->tc_ready) return KVR_ERR_UNSUPPORTED;
    cudaStream_t s = (cudaStream_t)stream_v;
    SetDevice sd(c->device);
    if (!sd.ok) return KVR_ERR_CUDA;

    // ---- plan: slots, shared-prefix dedupe, computed-token stream ----
    std::vector<int64_t> start(R + 1, 0);
    for (int r = 0; r < R; ++r) start[r + 1] = start[r] + lens[r];
    const int64_t T_in = start[R];
    c->last_slots.assign((size_t)T_in, -1);
    std::vector<int32_t> skip;
    plan_skips(lens, tables, valid_lens, R, width, B, c->keep_last != 0, skip);
    for (int r = 0; r < R; ++r)
        for (int t = 0; t < lens[r]; ++t)
            c->last_slots[(size_t)(start[r] + t)] = (int64_t)tables[(int64_t)r * width + t / B] * B + t % B;
    int64_t T = 0;
    for (int r = 0; r < R; ++r) T += lens[r] - skip[r];
    c->last_computed = T;
    c->have_last = false;
    c->dev_tables_current = false;
    c->last_chunks = 0;
    c->last_launches = 0;
    c->ev_kind.clear();
    if (T == 0) return KVR_OK;

    // computed stream -> chunks; attention tiles per chunk (longest context first)
    const int64_t Tc = c->max_chunk;
    const int64_t n_chunks = (T + Tc - 1) / Tc;
    std::vector<Chunk> chunks((size_t)n_chunks);
    for (int64_t k = 0; k < n_chunks; ++k) {
        chunks[k].off = k * Tc;
        chunks[k].n = (int32_t)std::min<int64_t>(Tc, T - k * Tc);
    }
    const size_t tables_bytes = (size_t)R * width * sizeof(int32_t);
    const size_t meta_bytes = (size_t)T * 4 * sizeof(int32_t);
    const size_t max_tiles_total = (size_t)(T / ATTN_TILE_Q + R + n_chunks + 1);
    const size_t tiles_bytes = align_up(max_tiles_total * sizeof(AttnTile));
    const size_t pairs_bytes = align_up((size_t)R * sizeof(int2));
    const size_t stage_bytes = align_up(tables_bytes) + align_up(meta_bytes) + tiles_bytes + pairs_bytes +
                               resume_meta_bytes(R);
    st = ensure_staging(c, stage_bytes);
    if (st != KVR_OK) return st;
    int32_t *st_tables = (int32_t *)c->pinned;
    int32_t *st_meta = (int32_t *)(c->pinned + align_up(tables_bytes));
    AttnTile *st_tiles = (AttnTile *)(c->pinned + align_up(tables_bytes) + align_up(meta_bytes));
    int2 *st_pairs = (int2 *)(c->pinned + align_up(tables_bytes) + align_up(meta_bytes) + tiles_bytes);
    std::vector<int32_t> pair_begin((size_t)n_chunks + 1, 0);
    size_t n_pairs = 0;
    std::memcpy(st_tables, tables, tables_bytes);
    {
        // chunk k's metadata block is [tok n][pos n][slot n][trow n] at st_meta + 4 * off
        int64_t g = 0;  // index in computed stream
        size_t n_tiles = 0;
        int64_t ck = 0;
        chunks[0].tile_begin = 0;
        for (int r = 0; r < R; ++r) {
            int32_t t = skip[r];
            while (t < lens[r]) {
                Chunk &ch = chunks[ck];
                const int64_t local = g - ch.off;
                const int32_t run = (int32_t)std::min<int64_t>(lens[r] - t, ch.n - local);
                int32_t *base = st_meta + 4 * ch.off;
                for (int32_t i = 0; i < run; ++i) {
                    const int32_t tt = t + i;
                    base[local + i] = tokens[start[r] + tt];
                    base[(int64_t)ch.n + local + i] = tt;
                    base[2 * (int64_t)ch.n + local + i] = tables[(int64_t)r * width + tt / B] * B + tt % B;
                    base[3 * (int64_t)ch.n + local + i] = r;
                }
                if (c->keep_last && t + run == lens[r]) st_pairs[n_pairs++] = make_int2((int)(local + run - 1), r);
                for (int32_t i = 0; i < run; i += tile_q) {
                    AttnTile &at = st_tiles[n_tiles++];
                    at.q_off = (int32_t)(local + i);
                    at.pos0 = t + i;
                    at.rows = std::min(tile_q, run - i);
                    at.trow = r;
                }
                g += run;
                t += run;
                if (g - ch.off == ch.n) {
                    pair_begin[ck + 1] = (int32_t)n_pairs;
                    ch.tile_end = (int32_t)n_tiles;
                    if (ck + 1 < n_chunks) chunks[ck + 1].tile_begin = (int32_t)n_tiles;
                    ++ck;
                }
            }
        }
        for (int64_t k = 0; k < n_chunks; ++k)
            std::stable_sort(st_tiles + chunks[k].tile_begin, st_tiles + chunks[k].tile_end,
                             [](const AttnTile &a, const AttnTile &b) { return a.pos0 + a.rows > b.pos0 + b.rows; });
    }

    // ---- enqueue ----
    char *ws = c->ws;
    const WsLayout &L = c->lay;
    float *h = (float *)(ws + L.h);
    void *a = ws + L.a;
    void *q = ws + L.q;
    void *m = ws + L.m;
    float2 *cs = (float2 *)(ws + L.cs);
    int32_t *d_meta = (int32_t *)(ws + L.meta);
    int32_t *d_tables = (int32_t *)(ws + L.tables);
    AttnTile *d_tiles = (AttnTile *)(ws + L.tiles);
    RopeFreq rf;
    for (int i = 0; i < md.hd / 2; ++i) rf.inv_freq[i] = std::pow(md.rope_base, -2.0 * i / md.hd);
    const size_t es = esize(c->desc.dtype);
    int64_t launches = 0;

    CU_OK(cudaMemcpyAsync(d_tables, st_tables, tables_bytes, cudaMemcpyHostToDevice, s));
    bool all_nonempty = true;
    for (int r = 0; r < R; ++r) all_nonempty = all_nonempty && lens[r] > 0;
    if (c->keep_last && all_nonempty) {
        // what kv_resume_logits needs besides the kept rows goes up with the tables
        char *st_resume = c->pinned + align_up(tables_bytes) + align_up(meta_bytes) + tiles_bytes + pairs_bytes;
        st = upload_resume_meta(c, st_resume, lens, R, s);
        if (st != KVR_OK) return st;
    }
    for (int64_t k = 0; k < n_chunks; ++k) {
        const Chunk &ch = chunks[k];
        const int n = ch.n;
        CU_OK(cudaMemcpyAsync(d_meta, st_meta + 4 * ch.off, (size_t)n * 4 * sizeof(int32_t),
                              cudaMemcpyHostToDevice, s));
        const int n_tiles = ch.tile_end - ch.tile_begin;
        if ((use_tc_attn || use_fa_attn) && n_tiles > 0)
            CU_OK(cudaMemcpyAsync(d_tiles, st_tiles + ch.tile_begin, (size_t)n_tiles * sizeof(AttnTile),
                                  cudaMemcpyHostToDevice, s));
        ChunkMeta cm{d_meta, d_meta + n, d_meta + 2 * (int64_t)n, d_meta + 3 * (int64_t)n, n};
        const int np = pair_begin[k + 1] - pair_begin[k];
        int2 *d_pairs = (int2 *)(ws + L.l_pairs);
        if (np > 0)
            CU_OK(cudaMemcpyAsync(d_pairs, st_pairs + pair_begin[k], (size_t)np * sizeof(int2), cudaMemcpyHostToDevice, s));
        { Timed tm(c, 0, s); launch_rope_table(cm.pos, n, md.hd, rf, cs, s); } ++launches;
        // Tensor-parallel ranks: a row-parallel projection leaves a partial sum in `part`; once summed over
        // the ranks it is added to the residual by the norm kernel that follows (tp_pending: still to be added).
        const bool tp = c->tp_world > 1;
        float *part = (float *)(ws + L.part);
        bool tp_pending = false;
        auto tp_allreduce = [&]() -> int {
            return c->tp_allreduce(part, (int64_t)n * md.d, (void *)s, c->tp_user) == 0 ? KVR_OK : KVR_ERR_CUDA;
        };
        for (int l = 0; l < md.L; ++l) {
            const bool last = (l == md.L - 1);
            {
                Timed tm(c, l == 0 ? 1 : 2, s);
                if (l == 0) launch_embed_rmsnorm(fp32, c->embed, c->w[W_LN1][0], cm, h, a, md.d, md.eps, s);
                else if (tp_pending) launch_add_rmsnorm(fp32, h, h, part, 1, 0, c->w[W_LN1][l], a, n, md.d, md.eps, s);
                else launch_rmsnorm(fp32, h, c->w[W_LN1][l], a, n, md.d, md.eps, s);
                tp_pending = false;
            }
            ++launches;
            if (last && np > 0) {   // h entering the last layer, for the tokens that end a request
                launch_gather_rows(h, md.d, d_pairs, np, (float *)(ws + L.l_h), s);
                ++launches;
            }
            // QKV projection + RoPE + paged store (last layer: K/V only)
            const QkvExtras ex = qkv_extras(c, l);
            if (use_tc_qkv) {
                TcGemmEpilogue ep{};
                set_tc_extras(ep, ex, !last);
                ep.mode = TC_QKV; ep.M = n; ep.K = md.d;
                ep.q_out = (__nv_bfloat16 *)q; ep.rope_cs = cs; ep.slot = cm.slot;
                ep.arena_k = (__nv_bfloat16 *)c->av.base + (int64_t)l * c->av.layer_stride;
                ep.kv_stride = c->av.kv_stride;
                ep.n_kv_cols = md.kv_dim; ep.head_dim = md.hd;
                CUtensorMap tb[3];
                if (last) {
                    ep.n_q_cols = 0; ep.n_b = 2;
                    tb[0] = c->tm_w[W_WK][l]; tb[1] = c->tm_w[W_WV][l]; tb[2] = tb[1];
                    ep.b_rows[0] = md.kv_dim; ep.b_rows[1] = md.kv_dim; ep.b_rows[2] = 0;
                } else {
                    ep.n_q_cols = md.q_dim; ep.n_b = 3;
                    tb[0] = c->tm_w[W_WQ][l]; tb[1] = c->tm_w[W_WK][l]; tb[2] = c->tm_w[W_WV][l];
                    ep.b_rows[0] = md.q_dim; ep.b_rows[1] = md.kv_dim; ep.b_rows[2] = md.kv_dim;
                }
                ep.N = ep.n_q_cols + 2 * md.kv_dim;
                { Timed tm(c, 3, s); st = launch_gemm_tc(c->tm_a_d, tb, ep, c->d_status, c->n_sms, s, nullptr, c->gemm_impl == 2); }
                if (st != KVR_OK) return st;
                ++launches;
            } else {
                Timed tm(c, 3, s);
                const int ld = md.q_dim + 2 * md.kv_dim;
                float *tmp = (float *)m;
                if (!last) {
                    launch_gemm_simt(fp32, 0, a, md.d, c->w[W_WQ][l], nullptr, md.d, n, md.q_dim, md.d, tmp, ld, s);
                    ++launches;
                }
                launch_gemm_simt(fp32, 0, a, md.d, c->w[W_WK][l], nullptr, md.d, n, md.kv_dim, md.d, tmp + md.q_dim,
                                 ld, s);
                launch_gemm_simt(fp32, 0, a, md.d, c->w[W_WV][l], nullptr, md.d, n, md.kv_dim, md.d,
                                 tmp + md.q_dim + md.kv_dim, ld, s);
                launch_rope_scatter(fp32, tmp, ld, cs, cm, md, c->av, l, !last, q, ex, s);
                launches += 3;
            }
            if (last) break;
            // causal attention over the paged K/V just written (output into `a`)
            {
                Timed tm(c, 4, s);
                if (use_fa_attn) {
                    st = launch_attn_fa(c->tm_q, c->tm_kv, d_tiles, n_tiles, d_tables, width, md, c->av, l,
                                        (__nv_bfloat16 *)a, c->d_status, s);
                    if (st != KVR_OK) return st;
                } else if (use_tc_attn) {
                    st = launch_attn_tc((const __nv_bfloat16 *)q, d_tiles, n_tiles, d_tables, width, md, c->av, l,
                                        (__nv_bfloat16 *)a, c->d_status, s);
                    if (st != KVR_OK) return st;
                } else {
                    launch_attn_simt(fp32, q, cm, d_tables, width, md, c->av, l, a, s);
                }
            }
            ++launches;
            // output projection + residual
            if (use_tc_gemm) {
                TcGemmEpilogue ep{};
                ep.mode = tp ? TC_STORE_F32 : TC_RESID; ep.M = n; ep.N = md.d; ep.K = md.q_dim;
                ep.c_f32 = tp ? part : h; ep.ldc = md.d;
                ep.n_b = 1; ep.b_rows[0] = md.d;
                CUtensorMap tb[3] = {c->tm_w[W_WO][l], c->tm_w[W_WO][l], c->tm_w[W_WO][l]};
                { Timed tm(c, 5, s); st = launch_gemm_tc(c->tm_a_q, tb, ep, c->d_status, c->n_sms, s, tp ? nullptr : &c->tm_h, c->gemm_impl == 2); }
                if (st != KVR_OK) return st;
            } else {
                Timed tm(c, 5, s);
                launch_gemm_simt(fp32, tp ? 0 : 1, a, md.q_dim, c->w[W_WO][l], nullptr, md.q_dim, n, md.d, md.q_dim,
                                 tp ? part : h, md.d, s);
            }
            ++launches;
            if (tp) {
                if ((st = tp_allreduce()) != KVR_OK) return st;
                Timed tm(c, 2, s);
                launch_add_rmsnorm(fp32, h, h, part, 1, 0, c->w[W_LN2][l], a, n, md.d, md.eps, s);
            } else {
                Timed tm(c, 2, s);
                launch_rmsnorm(fp32, h, c->w[W_LN2][l], a, n, md.d, md.eps, s);
            }
            ++launches;
            // gate/up + SwiGLU, then down + residual
            if (use_tc_gemm) {
                TcGemmEpilogue ep{};
                ep.mode = TC_SWIGLU; ep.M = n; ep.N = 2 * md.F; ep.K = md.d;
                ep.out_bf16 = (__nv_bfloat16 *)m; ep.ld_out = md.F;
                ep.n_b = 2; ep.b_rows[0] = md.F; ep.b_rows[1] = md.F;
                CUtensorMap tb[3] = {c->tm_w[W_WG][l], c->tm_w[W_WU][l], c->tm_w[W_WU][l]};
                { Timed tm(c, 6, s); st = launch_gemm_tc(c->tm_a_d, tb, ep, c->d_status, c->n_sms, s, nullptr, c->gemm_impl == 2); }
                if (st != KVR_OK) return st;
                TcGemmEpilogue e2{};
                e2.mode = tp ? TC_STORE_F32 : TC_RESID; e2.M = n; e2.N = md.d; e2.K = md.F;
                e2.c_f32 = tp ? part : h; e2.ldc = md.d;
                e2.n_b = 1; e2.b_rows[0] = md.d;
                CUtensorMap tb2[3] = {c->tm_w[W_WD][l], c->tm_w[W_WD][l], c->tm_w[W_WD][l]};
                { Timed tm(c, 7, s); st = launch_gemm_tc(c->tm_m, tb2, e2, c->d_status, c->n_sms, s, tp ? nullptr : &c->tm_h, c->gemm_impl == 2); }
                if (st != KVR_OK) return st;
            } else {
                { Timed tm(c, 6, s);
                  launch_gemm_simt(fp32, 2, a, md.d, c->w[W_WG][l], c->w[W_WU][l], md.d, n, md.F, md.d, m, md.F, s); }
                { Timed tm(c, 7, s);
                  launch_gemm_simt(fp32, tp ? 0 : 1, m, md.F, c->w[W_WD][l], nullptr, md.F, n, md.d, md.F,
                                   tp ? part : h, md.d, s); }
            }
            launches += 2;
            if (tp) {   // summed over the ranks now, added to the residual by the next layer's norm
                if ((st = tp_allreduce()) != KVR_OK) return st;
                tp_pending = true;
            }
        }
    }
    CU_OK(cudaEventRecord(c->staging_free, s));
    c->staging_busy = true;
    c->last_chunks = n_chunks;
    c->last_launches = launches;
    c->dev_tables_current = true;
    if (c->keep_last) {
        c->have_last = all_nonempty;
        c->last_lens.assign(lens, lens + R);
        c->last_tables.assign(tables, tables + (size_t)R * width);
        c->last_width = width;
    }
    (void)es;
    if (cudaGetLastError() != cudaSuccess) return KVR_ERR_CUDA;
    return KVR_OK;
}

static int readback_common(kvr_ctx *c, int32_t layer, const int32_t *table, int32_t n, void *k_out, void *v_out,
                           bool to_host, cudaStream_t s) {
    if (!c || n < 0 || (n > 0 && (!table || !k_out || !v_out))) return KVR_ERR_INVALID_ARG;
    if (!c->arena_bound || !c->ws_bound) return KVR_ERR_NOT_BOUND;
    if (layer < 0 || layer >= c->geom.n_layers) return KVR_ERR_INVALID_ARG;
    if (n == 0) return KVR_OK;
    const int B = c->geom.block_size;
    const int need = (n + B - 1) / B;
    for (int j = 0; j < need; ++j) {
        if (table[j] == -1) return KVR_ERR_TABLE_TOO_SHORT;
        if (table[j] < 0 || table[j] >= c->geom.num_blocks) return KVR_ERR_BLOCK_OOB;
    }
    if (need > c->max_blk) return KVR_ERR_WORKSPACE;
    const size_t es = esize(c->geom.dtype);
    const size_t dense = (size_t)n * c->av.row * es;
    if (to_host && 2 * align_up(dense) > c->lay.m_bytes) return KVR_ERR_WORKSPACE;
    SetDevice sd(c->device);
    int st = ensure_staging(c, (size_t)need * sizeof(int32_t));
    if (st != KVR_OK) return st;
    std::memcpy(c->pinned, table, (size_t)need * sizeof(int32_t));
    int32_t *d_tab = (int32_t *)(c->ws + c->lay.tables);
    c->dev_tables_current = false;   // this call's table goes over them
    CU_OK(cudaMemcpyAsync(d_tab, c->pinned, (size_t)need * sizeof(int32_t), cudaMemcpyHostToDevice, s));
    CU_OK(cudaEventRecord(c->staging_free, s));
    c->staging_busy = true;
    const bool fp32 = c->geom.dtype == KVR_FP32;
    if (to_host) {
        char *stage_k = c->ws + c->lay.m, *stage_v = stage_k + align_up(dense);
        launch_readback(fp32, c->av, layer, d_tab, n, stage_k, stage_v, s);
        CU_OK(cudaMemcpyAsync(k_out, stage_k, dense, cudaMemcpyDeviceToHost, s));
        CU_OK(cudaMemcpyAsync(v_out, stage_v, dense, cudaMemcpyDeviceToHost, s));
        CU_OK(cudaStreamSynchronize(s));
    } else {
        launch_readback(fp32, c->av, layer, d_tab, n, k_out, v_out, s);
        if (cudaGetLastError() != cudaSuccess) return KVR_ERR_CUDA;
    }
    return KVR_OK;
}

int kv_readback(kvr_ctx *c, int32_t layer, const int32_t *table, int32_t n, void *k_out, void *v_out, void *s) {
    return readback_common(c, layer, table, n, k_out, v_out, true, (cudaStream_t)s);
}

int kv_readback_dev(kvr_ctx *c, int32_t layer, const int32_t *table, int32_t n, void *k_out, void *v_out,
                    void *s) {
    return readback_common(c, layer, table, n, k_out, v_out, false, (cudaStream_t)s);
}

int kv_sync_status(kvr_ctx *c, void *stream) {
    if (!c) return KVR_ERR_INVALID_ARG;
    SetDevice sd(c->device);
    if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return KVR_ERR_CUDA;
    int v = 0;
    if (cudaMemcpy(&v, c->d_status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return KVR_ERR_CUDA;
    if (v != 0) {
        cudaMemset(c->d_status, 0, sizeof(int));
        return KVR_ERR_DEVICE_TIMEOUT;
    }
    return KVR_OK;
}

int kv_resume_logits(kvr_ctx *c, const void *final_gain, const void *lm_head, float *logits_out, void *stream) {
    if (!c || !final_gain || !lm_head || !logits_out) return KVR_ERR_INVALID_ARG;
    if (!c->arena_bound || !c->weights_bound || !c->ws_bound) return KVR_ERR_NOT_BOUND;
    if (!c->have_last) return KVR_ERR_NOT_BOUND;   // no rebuild with "keep_last_hidden" came before
    const ModelDims &md = c->md;
    const bool fp32 = is_fp32(c);
    const bool use_tc = !fp32 && c->gemm_impl >= 1;
    const bool use_tc_q = use_tc && md.q_dim % 128 == 0;   // as in the rebuild: whole 128-column halves only
    const bool use_fa = !fp32 && c->attn_impl >= 2 && c->tm_kv_ok;   // one-row tiles: the single-CTA kernel
    const bool use_mma = !fp32 && !use_fa && c->attn_impl != 0;
    if ((use_tc || use_fa || use_mma) && !c->tc_ready) return KVR_ERR_UNSUPPORTED;
    if ((((uintptr_t)lm_head) % 16) || (((uintptr_t)final_gain) % 16)) return KVR_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    SetDevice sd(c->device);
    const int R = (int)c->last_lens.size(), width = c->last_width, l = md.L - 1;
    char *ws = c->ws;
    const WsLayout &L = c->lay;
    // the rows the rebuild kept stay as they are (the call can be repeated); h is this call's residual
    const float *h0 = (const float *)(ws + L.l_h);
    float *h = (float *)(ws + L.l_h2);
    float *sk = (float *)(ws + L.l_sk);
    void *a = ws + L.l_a, *q = ws + L.l_q, *m = ws + L.l_m;
    float2 *cs = (float2 *)(ws + L.l_cs);
    int32_t *d_pos = (int32_t *)(ws + L.l_pos), *d_row = d_pos + R;
    int32_t *d_tables = (int32_t *)(ws + L.tables);
    AttnTile *d_tiles = (AttnTile *)(ws + L.l_tiles);
    // the block tables and the per-request metadata are still in the workspace when nothing but the rebuild
    // has used it since; otherwise they go up again
    int st = KVR_OK;
    if (!c->dev_tables_current) {
        const size_t tb = (size_t)R * width * sizeof(int32_t);
        st = ensure_staging(c, align_up(tb) + resume_meta_bytes(R));
        if (st != KVR_OK) return st;
        std::memcpy(c->pinned, c->last_tables.data(), tb);
        CU_OK(cudaMemcpyAsync(d_tables, c->pinned, tb, cudaMemcpyHostToDevice, s));
        st = upload_resume_meta(c, c->pinned + align_up(tb), c->last_lens.data(), R, s);
        if (st != KVR_OK) return st;
        CU_OK(cudaEventRecord(c->staging_free, s));
        c->staging_busy = true;
        c->dev_tables_current = true;
    }
    RopeFreq rf;
    for (int i = 0; i < md.hd / 2; ++i) rf.inv_freq[i] = std::pow(md.rope_base, -2.0 * i / md.hd);
    ChunkMeta cm{d_pos, d_pos, d_pos, d_row, R};   // tok and slot are not used on this path
    launch_rope_table(d_pos, R, md.hd, rf, cs, s);
    // few rows: every projection is bound by reading its weights once, which the weight-streaming GEMM does
    // on all SMs; its K splits leave fp32 partial products that the next kernel sums
    const bool use_sk = use_tc && c->resume_gemm == 1 && R <= GEMM_SKINNY_MAX_ROWS;
    // on that path every kernel after the first norm may be scheduled while the one before it drains
    // Tensor-parallel ranks: the output and down projections leave this rank's partial sums in `sk`, the callback
    // sums them over the ranks, the norm that follows adds them to the residual; the head is whole on every rank.
    const bool tp = c->tp_world > 1;
    auto tp_sum = [&](int64_t count) -> int {
        if (!tp) return KVR_OK;
        return c->tp_allreduce(sk, count, (void *)s, c->tp_user) == 0 ? KVR_OK : KVR_ERR_CUDA;
    };
    const bool pdl = use_sk && c->resume_pdl && !tp;   // the callback's work sits between the kernels of the chain
    if (!use_sk) CU_OK(cudaMemcpyAsync(h, h0, (size_t)R * md.d * sizeof(float), cudaMemcpyDeviceToDevice, s));
    launch_rmsnorm(fp32, h0, c->w[W_LN1][l], a, R, md.d, md.eps, s);
    // q of the final tokens (RoPE at position len - 1); their K/V are already in the arena
    QkvExtras ex = qkv_extras(c, l);
    ex.bk = ex.bv = ex.kn = nullptr;   // only q is projected here
    ModelDims q_only = md;
    q_only.Hkv = 0; q_only.kv_dim = 0;
    if (use_sk) {
        const int sp = gemm_skinny_splits(md.q_dim, md.d, c->n_sms);
        SkinnyArgs ga{};
        ga.R = R; ga.N = md.q_dim; ga.K = md.d; ga.out_f32 = sk; ga.split_stride = (int64_t)R * md.q_dim;
        ga.ldo = md.q_dim;
        st = launch_gemm_skinny(c->tm_x_d, c->tm_w[W_WQ][l], nullptr, ga, c->x_rows, sp, c->d_status, c->n_sms, s, pdl);
        if (st != KVR_OK) return st;
        launch_rope_scatter(false, sk, md.q_dim, cs, cm, q_only, c->av, l, true, q, ex, s, sp, ga.split_stride, pdl);
    } else if (use_tc_q) {
        TcGemmEpilogue ep{};
        set_tc_extras(ep, ex, true);
        ep.mode = TC_QKV; ep.M = R; ep.K = md.d; ep.N = md.q_dim;
        ep.q_out = (__nv_bfloat16 *)q; ep.rope_cs = cs; ep.slot = d_pos;
        ep.arena_k = (__nv_bfloat16 *)c->av.base; ep.kv_stride = 0;
        ep.n_q_cols = md.q_dim; ep.n_kv_cols = 0; ep.head_dim = md.hd;
        ep.n_b = 1; ep.b_rows[0] = md.q_dim;
        CUtensorMap tbm[3] = {c->tm_w[W_WQ][l], c->tm_w[W_WQ][l], c->tm_w[W_WQ][l]};
        st = launch_gemm_tc(c->tm_la_d, tbm, ep, c->d_status, c->n_sms, s, nullptr, c->gemm_impl == 2);
        if (st != KVR_OK) return st;
    } else {
        float *tmp = (float *)m;
        launch_gemm_simt(fp32, 0, a, md.d, c->w[W_WQ][l], nullptr, md.d, R, md.q_dim, md.d, tmp, md.q_dim, s);
        launch_rope_scatter(fp32, tmp, md.q_dim, cs, cm, q_only, c->av, l, true, q, ex, s);
    }
    // one query row per request: the split-KV kernel reads each request's K/V once (bf16, groups of up to 8 heads)
    const bool use_decode = !fp32 && c->attn_impl != 0 && md.Hq / md.Hkv <= 8;
    if (use_decode) {
        int max_len = 0;
        for (int r = 0; r < R; ++r) max_len = std::max(max_len, c->last_lens[r]);
        st = launch_attn_decode((const __nv_bfloat16 *)q, d_pos, R, max_len, d_tables, width, md, c->av, l,
                                (float *)(ws + L.l_part), (__nv_bfloat16 *)a, s, pdl);
        if (st != KVR_OK) return st;
    } else if (use_fa) {
        st = launch_attn_fa(c->tm_lq, c->tm_kv, d_tiles, R, d_tables, width, md, c->av, l, (__nv_bfloat16 *)a,
                            c->d_status, s);
        if (st != KVR_OK) return st;
    } else if (use_mma) {
        st = launch_attn_tc((const __nv_bfloat16 *)q, d_tiles, R, d_tables, width, md, c->av, l, (__nv_bfloat16 *)a,
                            c->d_status, s);
        if (st != KVR_OK) return st;
    } else {
        launch_attn_simt(fp32, q, cm, d_tables, width, md, c->av, l, a, s);
    }
    if (use_sk) {
        // output projection -> h = h0 + o Wo^T, norm; SwiGLU pair; down projection -> h += ..., final norm; head
        const int64_t hs = (int64_t)R * md.d;
        int sp = gemm_skinny_splits(md.d, md.q_dim, c->n_sms);
        SkinnyArgs go{};
        go.R = R; go.N = md.d; go.K = md.q_dim; go.out_f32 = sk; go.split_stride = hs; go.ldo = md.d;
        st = launch_gemm_skinny(c->tm_x_q, c->tm_w[W_WO][l], nullptr, go, c->x_rows, sp, c->d_status, c->n_sms, s, pdl);
        if (st != KVR_OK) return st;
        if ((st = tp_sum(sp * hs)) != KVR_OK) return st;
        launch_add_rmsnorm(false, h0, h, sk, sp, hs, c->w[W_LN2][l], a, R, md.d, md.eps, s, pdl);
        SkinnyArgs gg{};
        gg.R = R; gg.N = md.F; gg.K = md.d; gg.out_bf16 = (__nv_bfloat16 *)m; gg.ld_bf16 = md.F;
        st = launch_gemm_skinny(c->tm_x_d, c->tm_w[W_WG][l], &c->tm_w[W_WU][l], gg, c->x_rows, 1, c->d_status, c->n_sms, s, pdl);
        if (st != KVR_OK) return st;
        sp = gemm_skinny_splits(md.d, md.F, c->n_sms);
        SkinnyArgs gd{};
        gd.R = R; gd.N = md.d; gd.K = md.F; gd.out_f32 = sk; gd.split_stride = hs; gd.ldo = md.d;
        st = launch_gemm_skinny(c->tm_x_m, c->tm_w[W_WD][l], nullptr, gd, c->x_rows, sp, c->d_status, c->n_sms, s, pdl);
        if (st != KVR_OK) return st;
        if ((st = tp_sum(sp * hs)) != KVR_OK) return st;
        launch_add_rmsnorm(false, h, h, sk, sp, hs, final_gain, a, R, md.d, md.eps, s, pdl);
        CUtensorMap tlm;
        st = tc_make_tmap_2d(&tlm, lm_head, md.V, md.d, 128, 64);
        if (st != KVR_OK) return st;
        SkinnyArgs gl{};
        gl.R = R; gl.N = md.V; gl.K = md.d; gl.out_f32 = logits_out; gl.split_stride = 0; gl.ldo = md.V;
        st = launch_gemm_skinny(c->tm_x_d, tlm, nullptr, gl, c->x_rows, 1, c->d_status, c->n_sms, s, pdl);
        if (st != KVR_OK) return st;
        return cudaGetLastError() == cudaSuccess ? KVR_OK : KVR_ERR_CUDA;
    }
    const int64_t hs = (int64_t)R * md.d;
    if (use_tc) {
        TcGemmEpilogue ep{};
        ep.mode = tp ? TC_STORE_F32 : TC_RESID; ep.M = R; ep.N = md.d; ep.K = md.q_dim; ep.c_f32 = tp ? sk : h;
        ep.ldc = md.d;
        ep.n_b = 1; ep.b_rows[0] = md.d;
        CUtensorMap tbm[3] = {c->tm_w[W_WO][l], c->tm_w[W_WO][l], c->tm_w[W_WO][l]};
        st = launch_gemm_tc(c->tm_la_q, tbm, ep, c->d_status, c->n_sms, s, tp ? nullptr : &c->tm_lh, c->gemm_impl == 2);
        if (st != KVR_OK) return st;
    } else {
        launch_gemm_simt(fp32, tp ? 0 : 1, a, md.q_dim, c->w[W_WO][l], nullptr, md.q_dim, R, md.d, md.q_dim,
                         tp ? sk : h, md.d, s);
    }
    if (tp) {
        if ((st = tp_sum(hs)) != KVR_OK) return st;
        launch_add_rmsnorm(fp32, h, h, sk, 1, 0, c->w[W_LN2][l], a, R, md.d, md.eps, s);
    } else {
        launch_rmsnorm(fp32, h, c->w[W_LN2][l], a, R, md.d, md.eps, s);
    }
    if (use_tc) {
        TcGemmEpilogue ep{};
        ep.mode = TC_SWIGLU; ep.M = R; ep.N = 2 * md.F; ep.K = md.d;
        ep.out_bf16 = (__nv_bfloat16 *)m; ep.ld_out = md.F; ep.n_b = 2; ep.b_rows[0] = md.F; ep.b_rows[1] = md.F;
        CUtensorMap tbm[3] = {c->tm_w[W_WG][l], c->tm_w[W_WU][l], c->tm_w[W_WU][l]};
        st = launch_gemm_tc(c->tm_la_d, tbm, ep, c->d_status, c->n_sms, s, nullptr, c->gemm_impl == 2);
        if (st != KVR_OK) return st;
        TcGemmEpilogue e2{};
        e2.mode = tp ? TC_STORE_F32 : TC_RESID; e2.M = R; e2.N = md.d; e2.K = md.F; e2.c_f32 = tp ? sk : h;
        e2.ldc = md.d;
        e2.n_b = 1; e2.b_rows[0] = md.d;
        CUtensorMap tb2[3] = {c->tm_w[W_WD][l], c->tm_w[W_WD][l], c->tm_w[W_WD][l]};
        st = launch_gemm_tc(c->tm_lm, tb2, e2, c->d_status, c->n_sms, s, tp ? nullptr : &c->tm_lh, c->gemm_impl == 2);
        if (st != KVR_OK) return st;
    } else {
        launch_gemm_simt(fp32, 2, a, md.d, c->w[W_WG][l], c->w[W_WU][l], md.d, R, md.F, md.d, m, md.F, s);
        launch_gemm_simt(fp32, tp ? 0 : 1, m, md.F, c->w[W_WD][l], nullptr, md.F, R, md.d, md.F, tp ? sk : h, md.d, s);
    }
    // final norm and LM head
    if (tp) {
        if ((st = tp_sum(hs)) != KVR_OK) return st;
        launch_add_rmsnorm(fp32, h, h, sk, 1, 0, final_gain, a, R, md.d, md.eps, s);
    } else {
        launch_rmsnorm(fp32, h, final_gain, a, R, md.d, md.eps, s);
    }
    if (use_tc) {
        CUtensorMap tlm;
        st = tc_make_tmap_2d(&tlm, lm_head, md.V, md.d, 128, 64);
        if (st != KVR_OK) return st;
        TcGemmEpilogue ep{};
        ep.mode = TC_STORE_F32; ep.M = R; ep.N = md.V; ep.K = md.d; ep.c_f32 = logits_out; ep.ldc = md.V;
        ep.n_b = 1; ep.b_rows[0] = md.V;
        CUtensorMap tbm[3] = {tlm, tlm, tlm};
        st = launch_gemm_tc(c->tm_la_d, tbm, ep, c->d_status, c->n_sms, s, nullptr, c->gemm_impl == 2);
        if (st != KVR_OK) return st;
    } else {
        launch_gemm_simt(fp32, 0, a, md.d, lm_head, nullptr, md.d, R, md.V, md.d, logits_out, md.V, s);
    }
    return cudaGetLastError() == cudaSuccess ? KVR_OK : KVR_ERR_CUDA;
}

int kv_arena_flush(kvr_ctx *c, uint32_t fill_word, void *stream) {
    if (!c) return KVR_ERR_INVALID_ARG;
    if (!c->arena_bound) return KVR_ERR_NOT_BOUND;
    SetDevice sd(c->device);
    const size_t es = esize(c->geom.dtype);
    const size_t bytes = (size_t)c->geom.n_layers * (size_t)c->av.layer_stride * es;
    return launch_arena_flush(c->av.base, bytes, fill_word, c->n_sms, (cudaStream_t)stream);
}

int kv_health_probe(kvr_ctx *c, uint32_t seed, int32_t timeout_ms, uint32_t *checksum_out, void *stream) {
    if (!c || timeout_ms <= 0) return KVR_ERR_INVALID_ARG;
    SetDevice sd(c->device);
    cudaStream_t s = (cudaStream_t)stream;
    const int blocks = std::min(c->n_sms, (int)PROBE_MAX_BLOCKS);
    const long long limit = (long long)timeout_ms * (long long)std::max(c->clock_khz, 1000);   // cycles
    uint32_t *flags = c->d_probe, *out = c->d_probe + PROBE_MAX_BLOCKS;
    cudaEvent_t done;
    CU_OK(cudaEventCreateWithFlags(&done, cudaEventDisableTiming));
    if (++c->probe_epoch == 0) c->probe_epoch = 1;   // flags start at 0 and hold earlier epochs only
    int st = launch_probe(seed, c->probe_epoch, flags, out, c->d_status, blocks, limit, c->probe_mute ? 0 : 1, s);
    if (st == KVR_OK && cudaEventRecord(done, s) != cudaSuccess) st = KVR_ERR_CUDA;
    if (st == KVR_OK) {
        // host-side bound: the device waits give up after timeout_ms, so 2 x that is generous
        const auto t0 = std::chrono::steady_clock::now();
        cudaError_t q;
        while ((q = cudaEventQuery(done)) == cudaErrorNotReady) {
            if (std::chrono::steady_clock::now() - t0 > std::chrono::milliseconds(2 * (int64_t)timeout_ms + 50)) break;
            std::this_thread::sleep_for(std::chrono::microseconds(50));
        }
        if (q == cudaErrorNotReady) st = KVR_ERR_DEVICE_TIMEOUT;
        else if (q != cudaSuccess) st = KVR_ERR_CUDA;
    }
    cudaEventDestroy(done);
    if (st != KVR_OK) return st;
    int dev_status = 0;
    std::vector<uint32_t> res(blocks);
    CU_OK(cudaMemcpy(&dev_status, c->d_status, sizeof(int), cudaMemcpyDeviceToHost));
    CU_OK(cudaMemcpy(res.data(), out, blocks * sizeof(uint32_t), cudaMemcpyDeviceToHost));
    if (dev_status != 0) {
        cudaMemset(c->d_status, 0, sizeof(int));
        return KVR_ERR_DEVICE_TIMEOUT;
    }
    uint32_t sum = 0;
    for (int b = 0; b < blocks; ++b) {
        const int r = b & 31;
        sum ^= r ? ((res[b] << r) | (res[b] >> (32 - r))) : res[b];
    }
    if (checksum_out) *checksum_out = sum;
    return KVR_OK;
}

int kv_debug_slot_map(kvr_ctx *c, int64_t *out, int64_t n) {
    if (!c || !out || n < 0) return KVR_ERR_INVALID_ARG;
    if ((size_t)n != c->last_slots.size()) return KVR_ERR_INVALID_ARG;
    std::memcpy(out, c->last_slots.data(), (size_t)n * sizeof(int64_t));
    return KVR_OK;
}

int kv_debug_plan(kvr_ctx *c, int64_t *computed, int64_t *n_chunks, int64_t *n_launches) {
    if (!c) return KVR_ERR_INVALID_ARG;
    if (computed) *computed = c->last_computed;
    if (n_chunks) *n_chunks = c->last_chunks;
    if (n_launches) *n_launches = c->last_launches;
    return KVR_OK;
}

int kv_debug_profile(kvr_ctx *c, double *ms, int64_t *cnt) {
    if (!c || !ms || !cnt) return KVR_ERR_INVALID_ARG;
    SetDevice sd(c->device);
    for (int k = 0; k < KVR_N_KINDS; ++k) { ms[k] = 0.0; cnt[k] = 0; }
    for (size_t i = 0; i < c->ev_kind.size(); ++i) {
        if (cudaEventSynchronize(c->ev_pool[2 * i + 1]) != cudaSuccess) return KVR_ERR_CUDA;
        float t = 0.f;
        if (cudaEventElapsedTime(&t, c->ev_pool[2 * i], c->ev_pool[2 * i + 1]) != cudaSuccess) return KVR_ERR_CUDA;
        ms[c->ev_kind[i]] += t;
        cnt[c->ev_kind[i]] += 1;
    }
    return KVR_OK;
}

int kv_debug_gemm(kvr_ctx *c, int32_t impl, const void *a, const void *w, float *out, int32_t M, int32_t N,
                  int32_t K, void *stream) {
    if (!c || !a || !w || !out || M <= 0 || N <= 0 || K <= 0) return KVR_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    SetDevice sd(c->device);
    if (impl == 0) {
        launch_gemm_simt(false, 0, a, K, w, nullptr, K, M, N, K, out, N, s);
        return cudaGetLastError() == cudaSuccess ? KVR_OK : KVR_ERR_CUDA;
    }
    if (impl != 1 && impl != 2) return KVR_ERR_INVALID_ARG;
    if (!c->tc_ready) return KVR_ERR_UNSUPPORTED;
    if (K % 8 || ((uintptr_t)a) % 16 || ((uintptr_t)w) % 16) return KVR_ERR_UNSUPPORTED;
    CUtensorMap ta, tb[3];
    int st = tc_make_tmap_2d(&ta, a, M, K, 128, 64);
    if (st == KVR_OK) st = tc_make_tmap_2d(&tb[0], w, N, K, 128, 64);
    if (st != KVR_OK) return st;
    tb[1] = tb[0]; tb[2] = tb[0];
    TcGemmEpilogue ep{};
    ep.mode = TC_STORE_F32; ep.M = M; ep.N = N; ep.K = K; ep.c_f32 = out; ep.ldc = N; ep.n_b = 1; ep.b_rows[0] = N;
    return launch_gemm_tc(ta, tb, ep, c->d_status, c->n_sms, s, nullptr, impl == 2);
}

}  // extern "C"
