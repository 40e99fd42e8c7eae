// Attention for ONE query row per request (the final token of each logged prefix, used by
// kv_resume_logits): a recovered request needs its next-token logits after the arena is rebuilt
// (paper Sec. 4.2 step 5, Sec. 4.3).  With a single query row there is no matrix product worth a
// tensor-core tile; the step is bound by reading the request's K/V rows once.  So: the keys of a
// request are cut into splits, one CTA per (split, kv head, request) reads its K/V rows once for all
// query heads of the group (GQA), keeps a running softmax per head, and writes an unnormalised
// partial (max, sum, weighted values); a second small kernel merges the splits of every head.
// Both products run on warp-level MMAs in transposed form (keys, then head dims, as the rows of the tiles;
// the query heads of the group as the columns).
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

__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack2_bf16(float lo, float hi) {
    __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&h);
}

__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a) {
    uint32_t d;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
    return d;
}

// partial layout per (request, q head, split): [HD] weighted values, then max (log2 units) and sum
//
// Warp-level MMAs in the transposed form, so that no accumulator row is padding: per 32-key block of a warp
//   S^T = K Q^T   keys are the M dimension (two 16-key row tiles), the GQA group's heads the N dimension
//                 (G <= 8 columns; columns >= G see a zero Q).  The contraction runs over head dims, whose
//                 order is free as long as K and Q agree: lane c = lane % 4 takes dims 32 kp + 8 c .. + 7 of
//                 its two keys as ONE 16-byte load each and feeds them to k-steps 2 kp and 2 kp + 1.
//   softmax       a lane holds, for heads 2 c and 2 c + 1, the scores of keys g and g + 8 of each row tile;
//                 the column statistics are reduced over the eight lanes that share c.
//   O^T += V^T P^T   head dims are the M dimension (HD / 16 row tiles), heads the N dimension; P's accumulator
//                 fragments become B fragments by an 8 x 8 transpose across the warp (movmatrix); V rows go
//                 through shared memory (16-byte cp.async, XOR-swizzled) and ldmatrix.trans as A fragments.
template <int HD>
__global__ void __launch_bounds__(DEC_THREADS, 4)
attn_decode_partial_kernel(const __nv_bfloat16 *__restrict__ q, const int32_t *__restrict__ pos,
                           const int32_t *__restrict__ tables, int max_blk, int Hq, int Hkv,
                           const __nv_bfloat16 *__restrict__ arena_k, int64_t kv_stride, int block_size,
                           int split_len, int max_splits, float *__restrict__ partial) {
    constexpr int KP = HD / 32;            // 16-byte pieces of a key row per lane = pairs of k-steps of K Q^T
    constexpr int DT = HD / 16;            // 16-dim row tiles of O^T
    constexpr int ROW_CHUNKS = HD / 8;     // 16-byte chunks per V row
    grid_dependency_wait();
    grid_launch_dependents();
    const int sp = blockIdx.x, hk = blockIdx.y, r = blockIdx.z;
    const int G = Hq / Hkv;
    const int n_keys = pos[r] + 1;
    const int k0 = sp * split_len, k1 = min(n_keys, k0 + split_len);
    if (k0 >= k1) return;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, c = lane & 3;
    const int kv_dim = Hkv * HD, q_dim = Hq * HD;
    __shared__ __align__(16) __nv_bfloat16 vbuf[DEC_WARPS][32 * HD];
    __shared__ float red_m[DEC_WARPS][DEC_GMAX], red_l[DEC_WARPS][DEC_GMAX];
    // a warp's unnormalised output [G][HD] fp32 goes over its own V buffer once its key blocks are done
    static_assert(DEC_GMAX * HD * 4 <= 32 * HD * 2, "the V buffer holds a warp's partial output");
    const float scale_log2 = rsqrtf((float)HD) * 1.4426950408889634f;
    // Q^T fragments of head g (zero for g >= G): k-step 2 kp + ks uses dims 32 kp + 8 c + 4 ks + {0,1 | 2,3}
    uint32_t qb[2 * KP][2];
    {
        const uint2 *qrow = reinterpret_cast<const uint2 *>(q + (int64_t)r * q_dim + (hk * G + min(g, G - 1)) * HD);
#pragma unroll
        for (int kp = 0; kp < KP; ++kp)
#pragma unroll
            for (int ks = 0; ks < 2; ++ks) {
                const uint2 u = qrow[(32 * kp + 8 * c + 4 * ks) / 4];
                qb[2 * kp + ks][0] = g < G ? u.x : 0u;
                qb[2 * kp + ks][1] = g < G ? u.y : 0u;
            }
    }
    const int32_t *tab = tables + (int64_t)r * max_blk;
    const __nv_bfloat16 *arena_v = arena_k + kv_stride;
    const uint32_t vb = (uint32_t)__cvta_generic_to_shared(&vbuf[warp][0]);
    // running statistics of heads 2 c and 2 c + 1: the max is common to the eight lanes that share c, the sum
    // covers this lane's keys only (reduced over those lanes at the end)
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
    float o[DT][4];   // O^T: [0], [1] = dim 16 t + g of heads 2 c, 2 c + 1; [2], [3] = dim 16 t + g + 8
#pragma unroll
    for (int t = 0; t < DT; ++t) { o[t][0] = o[t][1] = o[t][2] = o[t][3] = 0.f; }
    for (int kb = k0 + warp * 32; kb < k1; kb += DEC_WARPS * 32) {
        // slot of key kb + lane (keys past the end borrow the last live key: finite rows, probability 0)
        const int key_l = min(kb + lane, k1 - 1);
        const int64_t slot_l = (int64_t)tab[key_l / block_size] * block_size + (key_l % block_size);
        // ---- V block -> shared memory, asynchronously (row = key, 16-byte chunk index XOR (key & 7)) ----
#pragma unroll
        for (int i = 0; i < 32 * ROW_CHUNKS / 32; ++i) {
            const int idx = i * 32 + lane, key = idx / ROW_CHUNKS, ch = idx % ROW_CHUNKS;
            const int64_t sl = __shfl_sync(0xffffffffu, slot_l, key);
            const __nv_bfloat16 *src = arena_v + sl * kv_dim + hk * HD + ch * 8;
            const uint32_t dst = vb + (uint32_t)(key * ROW_CHUNKS + (ch ^ (key & 7))) * 16u;
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
        // ---- S^T = K Q^T: two row tiles of 16 keys (rows g and g + 8 of each) ----
        float st[2][4];
        uint4 ka[2][KP], kc[2][KP];
#pragma unroll
        for (int mt = 0; mt < 2; ++mt) {
            const int64_t sa = __shfl_sync(0xffffffffu, slot_l, 16 * mt + g);
            const int64_t sc8 = __shfl_sync(0xffffffffu, slot_l, 16 * mt + g + 8);
            const uint4 *ra = reinterpret_cast<const uint4 *>(arena_k + sa * kv_dim + hk * HD);
            const uint4 *rc = reinterpret_cast<const uint4 *>(arena_k + sc8 * kv_dim + hk * HD);
#pragma unroll
            for (int kp = 0; kp < KP; ++kp) { ka[mt][kp] = ra[4 * kp + c]; kc[mt][kp] = rc[4 * kp + c]; }
        }
#pragma unroll
        for (int mt = 0; mt < 2; ++mt) {
            st[mt][0] = st[mt][1] = st[mt][2] = st[mt][3] = 0.f;
#pragma unroll
            for (int kp = 0; kp < KP; ++kp) {
                mma_bf16_16816(st[mt], ka[mt][kp].x, kc[mt][kp].x, ka[mt][kp].y, kc[mt][kp].y, qb[2 * kp][0],
                               qb[2 * kp][1]);
                mma_bf16_16816(st[mt], ka[mt][kp].z, kc[mt][kp].z, ka[mt][kp].w, kc[mt][kp].w, qb[2 * kp + 1][0],
                               qb[2 * kp + 1][1]);
            }
        }
        // ---- softmax statistics of heads 2 c, 2 c + 1 over the block's keys ----
        float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
        for (int mt = 0; mt < 2; ++mt)
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int key = kb + 16 * mt + g + 8 * (i >> 1);
                st[mt][i] = key < k1 ? st[mt][i] * scale_log2 : -INFINITY;
                mx[i & 1] = fmaxf(mx[i & 1], st[mt][i]);
            }
        float corr[2];
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            mx[e] = fmaxf(mx[e], __shfl_xor_sync(0xffffffffu, mx[e], 4));
            mx[e] = fmaxf(mx[e], __shfl_xor_sync(0xffffffffu, mx[e], 8));
            mx[e] = fmaxf(mx[e], __shfl_xor_sync(0xffffffffu, mx[e], 16));
            const float m_new = fmaxf(m_run[e], mx[e]);   // finite: the block has at least one live key
            corr[e] = ex2f(m_run[e] - m_new);
            m_run[e] = m_new;
        }
        uint32_t pb[2][2];   // P^T as B fragments of k-step mt: keys 16 mt + 2 c, + 1 | + 8, + 9 of head g
#pragma unroll
        for (int mt = 0; mt < 2; ++mt) {
            const float p0 = ex2f(st[mt][0] - m_run[0]), p1 = ex2f(st[mt][1] - m_run[1]);
            const float p2 = ex2f(st[mt][2] - m_run[0]), p3 = ex2f(st[mt][3] - m_run[1]);
            l_run[0] = (mt == 0 ? l_run[0] * corr[0] : l_run[0]) + p0 + p2;
            l_run[1] = (mt == 0 ? l_run[1] * corr[1] : l_run[1]) + p1 + p3;
            pb[mt][0] = movmatrix_trans(pack2_bf16(p0, p1));
            pb[mt][1] = movmatrix_trans(pack2_bf16(p2, p3));
        }
#pragma unroll
        for (int t = 0; t < DT; ++t) { o[t][0] *= corr[0]; o[t][1] *= corr[1]; o[t][2] *= corr[0]; o[t][3] *= corr[1]; }
        // ---- O^T += V^T P^T: two 16-key k-steps x DT row tiles; V^T fragments by ldmatrix.trans ----
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        __syncwarp();
#pragma unroll
        for (int mt = 0; mt < 2; ++mt) {
#pragma unroll
            for (int t = 0; t < DT; ++t) {
                // matrix j = lane / 8: keys 16 mt + 8 (j >> 1) + lane % 8, dims 16 t + 8 (j & 1) .. + 7
                const int j = lane >> 3, key = 16 * mt + 8 * (j >> 1) + (lane & 7), ch = 2 * t + (j & 1);
                const uint32_t addr = vb + (uint32_t)(key * ROW_CHUNKS + (ch ^ (key & 7))) * 16u;
                uint32_t a0, a1, a2, a3;
                asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                             : "=r"(a0), "=r"(a1), "=r"(a2), "=r"(a3) : "r"(addr));
                mma_bf16_16816(o[t], a0, a1, a2, a3, pb[mt][0], pb[mt][1]);
            }
        }
        __syncwarp();   // the V buffer is refilled at the top of the next block
    }
    // ---- merge the four warps (a warp that saw no key block has m = -inf, l = 0) ----
#pragma unroll
    for (int e = 0; e < 2; ++e) {
        l_run[e] += __shfl_xor_sync(0xffffffffu, l_run[e], 4);
        l_run[e] += __shfl_xor_sync(0xffffffffu, l_run[e], 8);
        l_run[e] += __shfl_xor_sync(0xffffffffu, l_run[e], 16);
    }
#pragma unroll
    for (int e = 0; e < 2; ++e) {
        const int hh = 2 * c + e;
        if (hh < G) {
            float *ro = reinterpret_cast<float *>(&vbuf[warp][0]) + hh * HD;
            if (g == 0) { red_m[warp][hh] = m_run[e]; red_l[warp][hh] = l_run[e]; }
#pragma unroll
            for (int t = 0; t < DT; ++t) {
                ro[16 * t + g] = o[t][e];
                ro[16 * t + g + 8] = o[t][2 + e];
            }
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < G * HD; i += DEC_THREADS) {
        const int gg = i / HD, d = i % HD;
        float M = -INFINITY;
        for (int w = 0; w < DEC_WARPS; ++w) M = fmaxf(M, red_m[w][gg]);
        float ov = 0.f, ls = 0.f;
        for (int w = 0; w < DEC_WARPS; ++w) {
            const float cw = red_m[w][gg] == -INFINITY ? 0.f : ex2f(red_m[w][gg] - M);
            ov = fmaf(cw, reinterpret_cast<const float *>(&vbuf[w][0])[gg * HD + d], ov);
            ls = fmaf(cw, red_l[w][gg], ls);
        }
        float *dst = partial + (((int64_t)r * Hq + hk * G + gg) * max_splits + sp) * (HD + 2);
        dst[d] = ov;
        if (d == 0) { dst[HD] = M; dst[HD + 1] = ls; }
    }
}

template <int HD>
__global__ void __launch_bounds__(HD)
attn_decode_merge_kernel(const float *__restrict__ partial, const int32_t *__restrict__ pos, int Hq, int split_len,
                         int max_splits, __nv_bfloat16 *__restrict__ o) {
    grid_dependency_wait();
    grid_launch_dependents();
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
                       __nv_bfloat16 *o, cudaStream_t s, bool pdl) {
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
        launch_kernel(attn_decode_partial_kernel<128>, grid, dim3(DEC_THREADS), 0, s, pdl, q, pos, tables, max_blk, md.Hq,
                      md.Hkv, ak, av.kv_stride, av.block_size, split_len, ATTN_DECODE_MAX_SPLITS, scratch);
        launch_kernel(attn_decode_merge_kernel<128>, mgrid, dim3(128), 0, s, pdl, (const float *)scratch, pos, md.Hq,
                      split_len, ATTN_DECODE_MAX_SPLITS, o);
    } else {
        launch_kernel(attn_decode_partial_kernel<64>, grid, dim3(DEC_THREADS), 0, s, pdl, q, pos, tables, max_blk, md.Hq,
                      md.Hkv, ak, av.kv_stride, av.block_size, split_len, ATTN_DECODE_MAX_SPLITS, scratch);
        launch_kernel(attn_decode_merge_kernel<64>, mgrid, dim3(64), 0, s, pdl, (const float *)scratch, pos, md.Hq,
                      split_len, ATTN_DECODE_MAX_SPLITS, o);
    }
    return cudaGetLastError() == cudaSuccess ? KVR_OK : KVR_ERR_CUDA;
}

}  // namespace kvr
