// Attention for ONE query row per request (the final token of each logged prefix, used by
// kv_resume_logits): a recovered request needs its next-token logits after the arena is rebuilt
// (paper Sec. 4.2 step 5, Sec. 4.3).  With a single query row there is no matrix product worth a
// tensor-core tile; the step is bound by reading the request's K/V rows once.  So: the keys of a
// request are cut into splits, one CTA per (split, kv head, request) reads its K/V rows once for all
// query heads of the group (GQA), keeps a running softmax per head, and writes an unnormalised
// partial (max, sum, weighted values); a second small kernel merges the splits of every head.
//   phase 1, lane = key:    scores of 32 keys against the group's query rows (q in shared memory)
//   phase 2, lane = dims:   the 32 probabilities (through shared memory) times the 32 value rows
#include "kvr_internal.h"

namespace kvr {

namespace {

constexpr int DEC_THREADS = 128, DEC_WARPS = 4, DEC_GMAX = 8;

__device__ __forceinline__ float ex2f(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ void bf16x8_to_f32(const uint4 &u, float (&f)[8]) {
    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        f[2 * i] = __uint_as_float(w[i] << 16);
        f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
}

// partial layout per (request, q head, split): [HD] weighted values, then max (log2 units) and sum
template <int HD>
__global__ void __launch_bounds__(DEC_THREADS)
attn_decode_partial_kernel(const __nv_bfloat16 *__restrict__ q, const int32_t *__restrict__ pos,
                           const int32_t *__restrict__ tables, int max_blk, int Hq, int Hkv,
                           const __nv_bfloat16 *__restrict__ arena_k, int64_t kv_stride, int block_size,
                           int split_len, int max_splits, float *__restrict__ partial) {
    constexpr int EPL = HD / 32;
    const int sp = blockIdx.x, hk = blockIdx.y, r = blockIdx.z;
    const int G = Hq / Hkv;
    const int n_keys = pos[r] + 1;
    const int k0 = sp * split_len, k1 = min(n_keys, k0 + split_len);
    if (k0 >= k1) return;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int kv_dim = Hkv * HD, q_dim = Hq * HD;
    __shared__ float qs[DEC_GMAX][HD];
    __shared__ float ps[DEC_WARPS][32][DEC_GMAX];
    __shared__ float red_o[DEC_WARPS][DEC_GMAX][HD];
    __shared__ float red_m[DEC_WARPS][DEC_GMAX], red_l[DEC_WARPS][DEC_GMAX];
    const float scale_log2 = rsqrtf((float)HD) * 1.4426950408889634f;
    for (int i = threadIdx.x; i < G * HD; i += DEC_THREADS) {
        const int g = i / HD, d = i % HD;
        qs[g][d] = __bfloat162float(q[(int64_t)r * q_dim + (hk * G + g) * HD + d]) * scale_log2;
    }
    __syncthreads();
    const int32_t *tab = tables + (int64_t)r * max_blk;
    float m[DEC_GMAX], l[DEC_GMAX], acc[DEC_GMAX][EPL];
#pragma unroll
    for (int g = 0; g < DEC_GMAX; ++g) {
        m[g] = -INFINITY;
        l[g] = 0.f;
#pragma unroll
        for (int e = 0; e < EPL; ++e) acc[g][e] = 0.f;
    }
    for (int kb = k0 + warp * 32; kb < k1; kb += DEC_WARPS * 32) {
        // ---- phase 1: lane = key ----
        const int key = kb + lane;
        const bool live = key < k1;
        int64_t slot = 0;
        float s[DEC_GMAX];
#pragma unroll
        for (int g = 0; g < DEC_GMAX; ++g) s[g] = 0.f;
        if (live) {
            slot = (int64_t)tab[key / block_size] * block_size + (key % block_size);
            const uint4 *kr = reinterpret_cast<const uint4 *>(arena_k + slot * kv_dim + hk * HD);
#pragma unroll 8
            for (int c = 0; c < HD / 8; ++c) {
                float kf[8];
                bf16x8_to_f32(kr[c], kf);
#pragma unroll
                for (int g = 0; g < DEC_GMAX; ++g) {
                    if (g < G) {
                        const float4 qa = *reinterpret_cast<const float4 *>(&qs[g][8 * c]);
                        const float4 qb = *reinterpret_cast<const float4 *>(&qs[g][8 * c + 4]);
                        s[g] = fmaf(qa.x, kf[0], fmaf(qa.y, kf[1], fmaf(qa.z, kf[2], fmaf(qa.w, kf[3], s[g]))));
                        s[g] = fmaf(qb.x, kf[4], fmaf(qb.y, kf[5], fmaf(qb.z, kf[6], fmaf(qb.w, kf[7], s[g]))));
                    }
                }
            }
        }
        float corr[DEC_GMAX];
#pragma unroll
        for (int g = 0; g < DEC_GMAX; ++g) {
            if (g < G) {
                float mx = live ? s[g] : -INFINITY;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
                const float mn = fmaxf(m[g], mx);            // finite: the block has at least one live key
                corr[g] = ex2f(m[g] - mn);
                const float p = live ? ex2f(s[g] - mn) : 0.f;
                l[g] = l[g] * corr[g] + p;                   // per-lane partial sums, reduced at the end
                m[g] = mn;
                ps[warp][lane][g] = p;
            }
        }
        __syncwarp();
        // ---- phase 2: lane = EPL dims ----
#pragma unroll
        for (int g = 0; g < DEC_GMAX; ++g)
            if (g < G) {
#pragma unroll
                for (int e = 0; e < EPL; ++e) acc[g][e] *= corr[g];
            }
        // All 32 keys of the block, eight value rows in flight at a time: a key past the end has
        // probability 0 and borrows the address of the block's last live key (its own slot may hold anything).
        const int n_live = min(32, k1 - kb);
#pragma unroll 8
        for (int kk = 0; kk < 32; ++kk) {
            const int64_t sl = __shfl_sync(0xffffffffu, slot, min(kk, n_live - 1));
            const __nv_bfloat16 *vr = arena_k + kv_stride + sl * kv_dim + hk * HD + lane * EPL;
            float vf[EPL];
            if (EPL == 4) {
                const uint2 u = *reinterpret_cast<const uint2 *>(vr);
                vf[0] = __uint_as_float(u.x << 16); vf[1] = __uint_as_float(u.x & 0xffff0000u);
                vf[2] = __uint_as_float(u.y << 16); vf[3] = __uint_as_float(u.y & 0xffff0000u);
            } else {
                const uint32_t u = *reinterpret_cast<const uint32_t *>(vr);
                vf[0] = __uint_as_float(u << 16); vf[1] = __uint_as_float(u & 0xffff0000u);
            }
#pragma unroll
            for (int g = 0; g < DEC_GMAX; ++g)
                if (g < G) {
                    const float p = ps[warp][kk][g];
#pragma unroll
                    for (int e = 0; e < EPL; ++e) acc[g][e] = fmaf(p, vf[e], acc[g][e]);
                }
        }
        __syncwarp();
    }
    // ---- merge the four warps (a warp that saw no key block has m = -inf, l = 0) ----
#pragma unroll
    for (int g = 0; g < DEC_GMAX; ++g)
        if (g < G) {
            float ls = l[g];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) ls += __shfl_xor_sync(0xffffffffu, ls, o);
            if (lane == 0) { red_m[warp][g] = m[g]; red_l[warp][g] = ls; }
#pragma unroll
            for (int e = 0; e < EPL; ++e) red_o[warp][g][lane * EPL + e] = acc[g][e];
        }
    __syncthreads();
    for (int i = threadIdx.x; i < G * HD; i += DEC_THREADS) {
        const int g = i / HD, d = i % HD;
        float M = -INFINITY;
        for (int w = 0; w < DEC_WARPS; ++w) M = fmaxf(M, red_m[w][g]);
        float o = 0.f, ls = 0.f;
        for (int w = 0; w < DEC_WARPS; ++w) {
            const float c = red_m[w][g] == -INFINITY ? 0.f : ex2f(red_m[w][g] - M);
            o = fmaf(c, red_o[w][g][d], o);
            ls = fmaf(c, red_l[w][g], ls);
        }
        float *dst = partial + (((int64_t)r * Hq + hk * G + g) * max_splits + sp) * (HD + 2);
        dst[d] = o;
        if (d == 0) { dst[HD] = M; dst[HD + 1] = ls; }
    }
}

template <int HD>
__global__ void __launch_bounds__(HD)
attn_decode_merge_kernel(const float *__restrict__ partial, const int32_t *__restrict__ pos, int Hq, int split_len,
                         int max_splits, __nv_bfloat16 *__restrict__ o) {
    const int hq = blockIdx.x, r = blockIdx.y, d = threadIdx.x;
    const int n_splits = (pos[r] + split_len) / split_len;   // ceil((pos + 1) / split_len)
    const float *base = partial + ((int64_t)r * Hq + hq) * max_splits * (HD + 2);
    float M = -INFINITY;
    for (int sp = 0; sp < n_splits; ++sp) M = fmaxf(M, base[sp * (HD + 2) + HD]);
    float acc = 0.f, ls = 0.f;
    for (int sp = 0; sp < n_splits; ++sp) {
        const float c = ex2f(base[sp * (HD + 2) + HD] - M);
        acc = fmaf(c, base[sp * (HD + 2) + d], acc);
        ls = fmaf(c, base[sp * (HD + 2) + HD + 1], ls);
    }
    o[(int64_t)r * Hq * HD + hq * HD + d] = __float2bfloat16(acc / ls);
}

}  // namespace

size_t attn_decode_scratch_bytes(int max_requests, int Hq, int hd) {
    return (size_t)max_requests * Hq * ATTN_DECODE_MAX_SPLITS * (hd + 2) * sizeof(float);
}

int launch_attn_decode(const __nv_bfloat16 *q, const int32_t *pos, int R, int max_len, const int32_t *tables,
                       int max_blk, const ModelDims &md, const ArenaView &av, int layer, float *scratch,
                       __nv_bfloat16 *o, cudaStream_t s) {
    if (R <= 0) return KVR_OK;
    if (md.Hq / md.Hkv > DEC_GMAX || (md.hd != 64 && md.hd != 128)) return KVR_ERR_UNSUPPORTED;
    // splits of at least 1024 keys, at most ATTN_DECODE_MAX_SPLITS per request, whole 32-key blocks
    int split_len = (max_len + ATTN_DECODE_MAX_SPLITS - 1) / ATTN_DECODE_MAX_SPLITS;
    split_len = split_len < 1024 ? 1024 : split_len;
    split_len = (split_len + 31) / 32 * 32;
    const int n_splits = (max_len + split_len - 1) / split_len;
    const __nv_bfloat16 *ak = (const __nv_bfloat16 *)av.base + (int64_t)layer * av.layer_stride;
    dim3 grid(n_splits, md.Hkv, R), mgrid(md.Hq, R);
    if (md.hd == 128) {
        attn_decode_partial_kernel<128><<<grid, DEC_THREADS, 0, s>>>(q, pos, tables, max_blk, md.Hq, md.Hkv, ak,
                                                                     av.kv_stride, av.block_size, split_len,
                                                                     ATTN_DECODE_MAX_SPLITS, scratch);
        attn_decode_merge_kernel<128><<<mgrid, 128, 0, s>>>(scratch, pos, md.Hq, split_len, ATTN_DECODE_MAX_SPLITS, o);
    } else {
        attn_decode_partial_kernel<64><<<grid, DEC_THREADS, 0, s>>>(q, pos, tables, max_blk, md.Hq, md.Hkv, ak,
                                                                    av.kv_stride, av.block_size, split_len,
                                                                    ATTN_DECODE_MAX_SPLITS, scratch);
        attn_decode_merge_kernel<64><<<mgrid, 64, 0, s>>>(scratch, pos, md.Hq, split_len, ATTN_DECODE_MAX_SPLITS, o);
    }
    return cudaGetLastError() == cudaSuccess ? KVR_OK : KVR_ERR_CUDA;
}

}  // namespace kvr
