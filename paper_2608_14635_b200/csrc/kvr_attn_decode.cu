// Attention for ONE query row per request (the final token of each logged prefix, used by
// kv_resume_logits): a recovered request needs its next-token logits after the arena is rebuilt
// (paper Sec. 4.2 step 5, Sec. 4.3).  With a single query row there is no matrix product worth a
// tensor-core tile; the step is bound by reading the request's K/V rows once.  So: the keys of a
// request are cut into splits, one CTA per (split, kv head, request) reads its K/V rows once for all
// query heads of the group (GQA), keeps a running softmax per head, and writes an unnormalised
// partial (max, sum, weighted values); a second small kernel merges the splits of every head.
// Both products run on warp-level MMAs with the query heads of the group as the rows of the tile.
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

// partial layout per (request, q head, split): [HD] weighted values, then max (log2 units) and sum
//
// Warp-level MMAs with the GQA group as the M dimension (rows 0..G-1 of a 16-row tile, G <= 8; rows
// 8..15 stay zero): per 32-key block of a warp
//   S = Q K^T   four 8-key column tiles x HD/16 k-steps.  The contraction runs over head dims, whose order
//               is free as long as Q and K agree: lane c = lane % 4 takes dims 32 kp + 8 c .. + 7 of its
//               key as ONE 16-byte load and feeds them to k-steps 2 kp and 2 kp + 1.
//   softmax     the accumulator fragment holds, for head lane / 4, the scores of keys 2 c, 2 c + 1 of each
//               column tile; row statistics are reduced over the four lanes of a row.
//   O += P V    P's accumulator fragments are already A fragments (two column tiles = one 16-key k-step); V
//               rows go through shared memory (16-byte cp.async, XOR-swizzled) and ldmatrix.trans.
template <int HD>
__global__ void __launch_bounds__(DEC_THREADS)
attn_decode_partial_kernel(const __nv_bfloat16 *__restrict__ q, const int32_t *__restrict__ pos,
                           const int32_t *__restrict__ tables, int max_blk, int Hq, int Hkv,
                           const __nv_bfloat16 *__restrict__ arena_k, int64_t kv_stride, int block_size,
                           int split_len, int max_splits, float *__restrict__ partial) {
    constexpr int KP = HD / 32;            // pairs of k-steps of Q K^T
    constexpr int NT = HD / 8;             // 8-dim column tiles of O
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
    // Q fragments of head g (zero rows for g >= G): k-step 2 kp + ks uses dims 32 kp + 8 c + 4 ks + {0,1 | 2,3}
    uint32_t qa[2 * KP][2];
    {
        const uint2 *qrow = reinterpret_cast<const uint2 *>(q + (int64_t)r * q_dim + (hk * G + min(g, G - 1)) * HD);
#pragma unroll
        for (int kp = 0; kp < KP; ++kp)
#pragma unroll
            for (int ks = 0; ks < 2; ++ks) {
                const uint2 u = qrow[(32 * kp + 8 * c + 4 * ks) / 4];
                qa[2 * kp + ks][0] = g < G ? u.x : 0u;
                qa[2 * kp + ks][1] = g < G ? u.y : 0u;
            }
    }
    const int32_t *tab = tables + (int64_t)r * max_blk;
    const __nv_bfloat16 *arena_v = arena_k + kv_stride;
    const uint32_t vb = (uint32_t)__cvta_generic_to_shared(&vbuf[warp][0]);
    float m_run = -INFINITY, l_run = 0.f;   // of head g, over this lane's keys (the sum is reduced over the row's lanes at the end)
    float o[NT][4];
#pragma unroll
    for (int t = 0; t < NT; ++t) { o[t][0] = o[t][1] = o[t][2] = o[t][3] = 0.f; }
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
        // ---- S = Q K^T: four column tiles of 8 keys ----
        float sacc[4][4];
#pragma unroll
        for (int t = 0; t < 4; ++t) {
            sacc[t][0] = sacc[t][1] = sacc[t][2] = sacc[t][3] = 0.f;
            const int64_t sl = __shfl_sync(0xffffffffu, slot_l, 8 * t + g);
            const uint4 *kr = reinterpret_cast<const uint4 *>(arena_k + sl * kv_dim + hk * HD);
            uint4 kf[KP];
#pragma unroll
            for (int kp = 0; kp < KP; ++kp) kf[kp] = kr[4 * kp + c];
#pragma unroll
            for (int kp = 0; kp < KP; ++kp) {
                mma_bf16_16816(sacc[t], qa[2 * kp][0], 0u, qa[2 * kp][1], 0u, kf[kp].x, kf[kp].y);
                mma_bf16_16816(sacc[t], qa[2 * kp + 1][0], 0u, qa[2 * kp + 1][1], 0u, kf[kp].z, kf[kp].w);
            }
        }
        // ---- softmax statistics of head g over the block's keys ----
        float sc[4][2], mx = -INFINITY;
#pragma unroll
        for (int t = 0; t < 4; ++t)
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int key = kb + 8 * t + 2 * c + e;
                sc[t][e] = key < k1 ? sacc[t][e] * scale_log2 : -INFINITY;
                mx = fmaxf(mx, sc[t][e]);
            }
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
        const float m_new = fmaxf(m_run, mx);          // finite: the block has at least one live key
        const float corr = ex2f(m_run - m_new);
        m_run = m_new;
        float ps = 0.f;
        uint32_t pa[4];                                // P as A fragments: tile t -> keys 8 t + 2 c, + 1
#pragma unroll
        for (int t = 0; t < 4; ++t) {
            const float p0 = ex2f(sc[t][0] - m_new), p1 = ex2f(sc[t][1] - m_new);
            ps += p0 + p1;
            pa[t] = pack2_bf16(p0, p1);
        }
        l_run = l_run * corr + ps;
#pragma unroll
        for (int t = 0; t < NT; ++t) { o[t][0] *= corr; o[t][1] *= corr; }
        // ---- O += P V: two 16-key k-steps x NT column tiles; V fragments by ldmatrix.trans ----
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        __syncwarp();
#pragma unroll
        for (int u = 0; u < 2; ++u) {
#pragma unroll
            for (int nt = 0; nt < NT; nt += 2) {
                // matrix j = lane / 8: keys 16 u + 8 (j & 1) + lane % 8, column tile nt + (j >> 1)
                const int j = lane >> 3, key = 16 * u + 8 * (j & 1) + (lane & 7), ch = nt + (j >> 1);
                const uint32_t addr = vb + (uint32_t)(key * ROW_CHUNKS + (ch ^ (key & 7))) * 16u;
                uint32_t b0, b1, b2, b3;
                asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                             : "=r"(b0), "=r"(b1), "=r"(b2), "=r"(b3) : "r"(addr));
                mma_bf16_16816(o[nt], pa[2 * u], 0u, pa[2 * u + 1], 0u, b0, b1);
                mma_bf16_16816(o[nt + 1], pa[2 * u], 0u, pa[2 * u + 1], 0u, b2, b3);
            }
        }
        __syncwarp();   // the V buffer is refilled at the top of the next block
    }
    // ---- merge the four warps (a warp that saw no key block has m = -inf, l = 0) ----
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
    if (g < G) {
        float *ro = reinterpret_cast<float *>(&vbuf[warp][0]) + g * HD;
        if (c == 0) { red_m[warp][g] = m_run; red_l[warp][g] = l_run; }
#pragma unroll
        for (int t = 0; t < NT; ++t) {
            ro[8 * t + 2 * c] = o[t][0];
            ro[8 * t + 2 * c + 1] = o[t][1];
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
