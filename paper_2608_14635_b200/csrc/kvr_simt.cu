// Plain-FMA kernels: embedding gather + RMSNorm, RMSNorm, RoPE table, a tiled
// fp32-accumulate GEMM, RoPE + paged K/V store, a warp-per-row causal attention
// over paged K/V, and the read-back gather.  They are the fp32 correctness mode
// and the memory-bound steps of the bf16 mode.
#include "kvr_internal.h"

namespace kvr {

template <typename T> __device__ __forceinline__ float to_f(T x);
template <> __device__ __forceinline__ float to_f<float>(float x) { return x; }
template <> __device__ __forceinline__ float to_f<__nv_bfloat16>(__nv_bfloat16 x) { return __bfloat162float(x); }
template <typename T> __device__ __forceinline__ T from_f(float x);
template <> __device__ __forceinline__ float from_f<float>(float x) { return x; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Sum over the block; every thread gets the result.  blockDim.x multiple of 32, <= 1024.
__device__ __forceinline__ float block_sum(float v, float *red) {
    v = warp_sum(v);
    const int w = threadIdx.x >> 5, l = threadIdx.x & 31, nw = blockDim.x >> 5;
    if (l == 0) red[w] = v;
    __syncthreads();
    float t = (l < nw) ? red[l] : 0.f;
    t = warp_sum(t);
    __syncthreads();
    return t;
}

// ---------------------------------------------------------------------------
// Embedding gather + input RMSNorm of layer 0: h = E[tok] (fp32), a = norm(h) g.
// One block per token; the row is held in shared memory between the two passes.
// ---------------------------------------------------------------------------
template <typename T, int VEC>
__device__ __forceinline__ void load_vec(const T *p, float (&v)[VEC]);
template <> __device__ __forceinline__ void load_vec<float, 4>(const float *p, float (&v)[4]) {
    float4 x = *reinterpret_cast<const float4 *>(p);
    v[0] = x.x; v[1] = x.y; v[2] = x.z; v[3] = x.w;
}
template <> __device__ __forceinline__ void load_vec<__nv_bfloat16, 8>(const __nv_bfloat16 *p, float (&v)[8]) {
    uint4 x = *reinterpret_cast<const uint4 *>(p);
    const __nv_bfloat162 *h = reinterpret_cast<const __nv_bfloat162 *>(&x);
#pragma unroll
    for (int i = 0; i < 4; ++i) { float2 f = __bfloat1622float2(h[i]); v[2 * i] = f.x; v[2 * i + 1] = f.y; }
}
template <> __device__ __forceinline__ void load_vec<__nv_bfloat16, 4>(const __nv_bfloat16 *p, float (&v)[4]) {
    uint2 x = *reinterpret_cast<const uint2 *>(p);
    const __nv_bfloat162 *h = reinterpret_cast<const __nv_bfloat162 *>(&x);
#pragma unroll
    for (int i = 0; i < 2; ++i) { float2 f = __bfloat1622float2(h[i]); v[2 * i] = f.x; v[2 * i + 1] = f.y; }
}
template <typename T, int VEC>
__device__ __forceinline__ void store_vec(T *p, const float (&v)[VEC]);
template <> __device__ __forceinline__ void store_vec<float, 4>(float *p, const float (&v)[4]) {
    *reinterpret_cast<float4 *>(p) = make_float4(v[0], v[1], v[2], v[3]);
}
template <> __device__ __forceinline__ void store_vec<__nv_bfloat16, 4>(__nv_bfloat16 *p, const float (&v)[4]) {
    uint2 x;
    __nv_bfloat162 *h = reinterpret_cast<__nv_bfloat162 *>(&x);
    h[0] = __floats2bfloat162_rn(v[0], v[1]);
    h[1] = __floats2bfloat162_rn(v[2], v[3]);
    *reinterpret_cast<uint2 *>(p) = x;
}
template <> __device__ __forceinline__ void store_vec<__nv_bfloat16, 8>(__nv_bfloat16 *p, const float (&v)[8]) {
    uint4 x;
    __nv_bfloat162 *h = reinterpret_cast<__nv_bfloat162 *>(&x);
#pragma unroll
    for (int i = 0; i < 4; ++i) h[i] = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
    *reinterpret_cast<uint4 *>(p) = x;
}

// d must be a multiple of VEC (host checks d % 8 == 0).
template <typename T, bool EMBED>
__global__ void __launch_bounds__(256) rmsnorm_kernel(const T *__restrict__ embed, const int32_t *__restrict__ tok,
                                                      float *__restrict__ h, const T *__restrict__ gain,
                                                      T *__restrict__ a, int d, float eps) {
    constexpr int VEC = sizeof(T) == 4 ? 4 : 8;
    extern __shared__ float row[];
    __shared__ float red[32];
    const int64_t t = blockIdx.x;
    float ss = 0.f;
    if (EMBED) {
        const T *src = embed + (int64_t)tok[t] * d;
        for (int i = threadIdx.x * VEC; i < d; i += blockDim.x * VEC) {
            float v[VEC];
            load_vec<T, VEC>(src + i, v);
#pragma unroll
            for (int j = 0; j < VEC; ++j) { row[i + j] = v[j]; ss += v[j] * v[j]; }
#pragma unroll
            for (int j = 0; j < VEC; j += 4)
                *reinterpret_cast<float4 *>(h + t * d + i + j) = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
        }
    } else {
        const float *src = h + t * d;
        for (int i = threadIdx.x * 4; i < d; i += blockDim.x * 4) {
            float4 x = *reinterpret_cast<const float4 *>(src + i);
            *reinterpret_cast<float4 *>(row + i) = x;
            ss += x.x * x.x + x.y * x.y + x.z * x.z + x.w * x.w;
        }
    }
    ss = block_sum(ss, red);
    const float rstd = 1.0f / sqrtf(ss / (float)d + eps);
    for (int i = threadIdx.x * VEC; i < d; i += blockDim.x * VEC) {
        float g[VEC], o[VEC];
        load_vec<T, VEC>(gain + i, g);
#pragma unroll
        for (int j = 0; j < VEC; ++j) o[j] = row[i + j] * rstd * g[j];
        store_vec<T, VEC>(a + t * d + i, o);
    }
}

// The same for rows already in h (every launch but the first of a chunk), with the row held in
// registers between the two passes: up to MAXV float4 per thread, i.e. d <= 1024 * MAXV.
template <typename T, int MAXV>
__global__ void __launch_bounds__(256) rmsnorm_reg_kernel(const float *__restrict__ h, const T *__restrict__ gain,
                                                          T *__restrict__ a, int d, float eps) {
    __shared__ float red[32];
    const int64_t t = blockIdx.x;
    const float *src = h + t * d;
    float4 x[MAXV];
    float ss = 0.f;
#pragma unroll
    for (int v = 0; v < MAXV; ++v) {
        const int i = (v * 256 + threadIdx.x) * 4;
        if (i < d) {
            x[v] = *reinterpret_cast<const float4 *>(src + i);
            ss += x[v].x * x[v].x + x[v].y * x[v].y + x[v].z * x[v].z + x[v].w * x[v].w;
        }
    }
    ss = block_sum(ss, red);
    const float rstd = 1.0f / sqrtf(ss / (float)d + eps);
#pragma unroll
    for (int v = 0; v < MAXV; ++v) {
        const int i = (v * 256 + threadIdx.x) * 4;
        if (i < d) {
            float g[4], o[4];
            load_vec<T, 4>(gain + i, g);
            o[0] = x[v].x * rstd * g[0];
            o[1] = x[v].y * rstd * g[1];
            o[2] = x[v].z * rstd * g[2];
            o[3] = x[v].w * rstd * g[3];
            store_vec<T, 4>(a + t * d + i, o);
        }
    }
}

// h_out = h_in + sum of n_part partial products (summed in index order), then the norm of the
// updated row.  Partial products come from the row-parallel projection of a tensor-parallel rank
// (one, already all-reduced) or from the K splits of the weight-streaming GEMM.
template <typename T>
__global__ void __launch_bounds__(256) add_rmsnorm_kernel(const float *__restrict__ h_in, float *__restrict__ h_out,
                                                          const float *__restrict__ part, int n_part,
                                                          int64_t part_stride, const T *__restrict__ gain,
                                                          T *__restrict__ a, int d, float eps) {
    constexpr int VEC = sizeof(T) == 4 ? 4 : 8;
    extern __shared__ float row[];
    __shared__ float red[32];
    grid_dependency_wait();
    grid_launch_dependents();
    const int64_t t = blockIdx.x;
    float ss = 0.f;
    for (int i = threadIdx.x * 4; i < d; i += blockDim.x * 4) {
        float4 x = *reinterpret_cast<const float4 *>(h_in + t * d + i);
        for (int p = 0; p < n_part; ++p) {
            const float4 y = *reinterpret_cast<const float4 *>(part + p * part_stride + t * d + i);
            x.x += y.x; x.y += y.y; x.z += y.z; x.w += y.w;
        }
        *reinterpret_cast<float4 *>(h_out + t * d + i) = x;
        *reinterpret_cast<float4 *>(row + i) = x;
        ss += x.x * x.x + x.y * x.y + x.z * x.z + x.w * x.w;
    }
    ss = block_sum(ss, red);
    const float rstd = 1.0f / sqrtf(ss / (float)d + eps);
    for (int i = threadIdx.x * VEC; i < d; i += blockDim.x * VEC) {
        float g[VEC], o[VEC];
        load_vec<T, VEC>(gain + i, g);
#pragma unroll
        for (int j = 0; j < VEC; ++j) o[j] = row[i + j] * rstd * g[j];
        store_vec<T, VEC>(a + t * d + i, o);
    }
}

void launch_add_rmsnorm(bool fp32, const float *h_in, float *h_out, const float *part, int n_part,
                        int64_t part_stride, const void *gain, void *a, int n, int d, float eps, cudaStream_t s,
                        bool pdl) {
    if (n == 0) return;
    const size_t sm = (size_t)d * sizeof(float);
    if (fp32)
        launch_kernel(add_rmsnorm_kernel<float>, dim3(n), dim3(256), sm, s, pdl, h_in, h_out, part, n_part, part_stride,
                      (const float *)gain, (float *)a, d, eps);
    else
        launch_kernel(add_rmsnorm_kernel<__nv_bfloat16>, dim3(n), dim3(256), sm, s, pdl, h_in, h_out, part, n_part,
                      part_stride, (const __nv_bfloat16 *)gain, (__nv_bfloat16 *)a, d, eps);
}

void launch_embed_rmsnorm(bool fp32, const void *embed, const void *gain, const ChunkMeta &cm, float *h,
                          void *a, int d, float eps, cudaStream_t s) {
    if (cm.n == 0) return;
    size_t sm = (size_t)d * sizeof(float);
    if (fp32)
        rmsnorm_kernel<float, true><<<cm.n, 256, sm, s>>>((const float *)embed, cm.tok, h, (const float *)gain,
                                                           (float *)a, d, eps);
    else
        rmsnorm_kernel<__nv_bfloat16, true><<<cm.n, 256, sm, s>>>((const __nv_bfloat16 *)embed, cm.tok, h,
                                                                   (const __nv_bfloat16 *)gain,
                                                                   (__nv_bfloat16 *)a, d, eps);
}

void launch_rmsnorm(bool fp32, const float *h, const void *gain, void *a, int n, int d, float eps,
                    cudaStream_t s) {
    if (n == 0) return;
    if (!fp32 && d % 4 == 0 && d <= 1024 * 6) {
        if (d <= 2048)
            rmsnorm_reg_kernel<__nv_bfloat16, 2><<<n, 256, 0, s>>>(h, (const __nv_bfloat16 *)gain, (__nv_bfloat16 *)a, d, eps);
        else if (d <= 4096)
            rmsnorm_reg_kernel<__nv_bfloat16, 4><<<n, 256, 0, s>>>(h, (const __nv_bfloat16 *)gain, (__nv_bfloat16 *)a, d, eps);
        else
            rmsnorm_reg_kernel<__nv_bfloat16, 6><<<n, 256, 0, s>>>(h, (const __nv_bfloat16 *)gain, (__nv_bfloat16 *)a, d, eps);
        return;
    }
    size_t sm = (size_t)d * sizeof(float);
    if (fp32)
        rmsnorm_kernel<float, false><<<n, 256, sm, s>>>(nullptr, nullptr, const_cast<float *>(h),
                                                         (const float *)gain, (float *)a, d, eps);
    else
        rmsnorm_kernel<__nv_bfloat16, false><<<n, 256, sm, s>>>(nullptr, nullptr, const_cast<float *>(h),
                                                                 (const __nv_bfloat16 *)gain,
                                                                 (__nv_bfloat16 *)a, d, eps);
}

// ---------------------------------------------------------------------------
// cos/sin of pos * base^(-2i/hd), evaluated in double, stored as float2.
// ---------------------------------------------------------------------------
__global__ void rope_table_kernel(const int32_t *__restrict__ pos, int n, int half, RopeFreq f,
                                  float2 *__restrict__ cs) {
    const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (int64_t)n * half) return;
    const int t = (int)(idx / half), i = (int)(idx % half);
    double sn, c;
    sincos((double)pos[t] * f.inv_freq[i], &sn, &c);
    cs[idx] = make_float2((float)c, (float)sn);
}

void launch_rope_table(const int32_t *pos, int n, int hd, const RopeFreq &f, float2 *cs, cudaStream_t s) {
    if (n == 0) return;
    const int half = hd / 2;
    const int64_t total = (int64_t)n * half;
    rope_table_kernel<<<(unsigned)((total + 255) / 256), 256, 0, s>>>(pos, n, half, f, cs);
}

// ---------------------------------------------------------------------------
// Tiled GEMM, fp32 accumulate in a fixed k order: C = A[M,K] W[N,K]^T.
// 64x64 tile, 16-wide k slab, 256 threads x (4x4) outputs.
// ---------------------------------------------------------------------------
template <typename T, int MODE>
__global__ void __launch_bounds__(256) gemm_simt_kernel(const T *__restrict__ A, int lda, const T *__restrict__ W0,
                                                        const T *__restrict__ W1, int ldw, int M, int N, int K,
                                                        void *__restrict__ Cv, int ldc) {
    constexpr int BM = 64, BN = 64, BK = 16;
    __shared__ float As[BK][BM + 4];
    __shared__ float Ws[BK][BN + 4];
    __shared__ float Us[MODE == 2 ? BK : 1][BN + 4];
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
    float acc[4][4] = {}, acc2[4][4] = {};
    for (int k0 = 0; k0 < K; k0 += BK) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int idx = threadIdx.x + i * 256;
            const int r = idx >> 4, k = idx & 15;
            const int gm = m0 + r, gn = n0 + r, gk = k0 + k;
            As[k][r] = (gm < M && gk < K) ? to_f<T>(A[(int64_t)gm * lda + gk]) : 0.f;
            Ws[k][r] = (gn < N && gk < K) ? to_f<T>(W0[(int64_t)gn * ldw + gk]) : 0.f;
            if (MODE == 2) Us[k][r] = (gn < N && gk < K) ? to_f<T>(W1[(int64_t)gn * ldw + gk]) : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < BK; ++k) {
            float a[4], w[4], u[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) { a[i] = As[k][ty * 4 + i]; w[i] = Ws[k][tx * 4 + i]; }
            if (MODE == 2) {
#pragma unroll
                for (int i = 0; i < 4; ++i) u[i] = Us[k][tx * 4 + i];
            }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    acc[i][j] = fmaf(a[i], w[j], acc[i][j]);
                    if (MODE == 2) acc2[i][j] = fmaf(a[i], u[j], acc2[i][j]);
                }
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int gm = m0 + ty * 4 + i;
        if (gm >= M) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int gn = n0 + tx * 4 + j;
            if (gn >= N) continue;
            const int64_t o = (int64_t)gm * ldc + gn;
            if (MODE == 0) {
                ((float *)Cv)[o] = acc[i][j];
            } else if (MODE == 1) {
                ((float *)Cv)[o] += acc[i][j];
            } else {
                const float g = acc[i][j];
                ((T *)Cv)[o] = from_f<T>(g / (1.0f + expf(-g)) * acc2[i][j]);
            }
        }
    }
}

template <typename T>
static void gemm_simt_dispatch(int mode, const void *A, int lda, const void *W0, const void *W1, int ldw, int M,
                               int N, int K, void *C, int ldc, cudaStream_t s) {
    dim3 grid((N + 63) / 64, (M + 63) / 64);
    if (mode == 0)
        gemm_simt_kernel<T, 0><<<grid, 256, 0, s>>>((const T *)A, lda, (const T *)W0, nullptr, ldw, M, N, K, C, ldc);
    else if (mode == 1)
        gemm_simt_kernel<T, 1><<<grid, 256, 0, s>>>((const T *)A, lda, (const T *)W0, nullptr, ldw, M, N, K, C, ldc);
    else
        gemm_simt_kernel<T, 2><<<grid, 256, 0, s>>>((const T *)A, lda, (const T *)W0, (const T *)W1, ldw, M, N, K, C,
                                                     ldc);
}

void launch_gemm_simt(bool fp32, int mode, const void *A, int lda, const void *W0, const void *W1, int ldw,
                      int M, int N, int K, void *C, int ldc, cudaStream_t s) {
    if (M == 0 || N == 0) return;
    if (fp32) gemm_simt_dispatch<float>(mode, A, lda, W0, W1, ldw, M, N, K, C, ldc, s);
    else gemm_simt_dispatch<__nv_bfloat16>(mode, A, lda, W0, W1, ldw, M, N, K, C, ldc, s);
}

// ---------------------------------------------------------------------------
// RoPE + paged store.  One block per token.  Input: raw projections fp32
// [n, q_dim + 2 kv_dim] (q | k | v).  Q rotated -> q_out; K rotated and V raw ->
// arena rows at slot[t].
// ---------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(128) rope_scatter_kernel(const float *__restrict__ qkv, int ld, int n_part,
                                                           int64_t part_stride, const float2 *__restrict__ cs,
                                                           const int32_t *__restrict__ slot, int Hq, int Hkv, int hd,
                                                           T *__restrict__ arena_k, int64_t kv_stride,
                                                           bool want_q, T *__restrict__ q_out, QkvExtras ex) {
    grid_dependency_wait();
    grid_launch_dependents();
    const int64_t t = blockIdx.x;
    const int half = hd >> 1;
    const float *src0 = qkv + t * ld;
    // the projection may arrive as n_part partial products (K splits), summed here in index order
    auto src = [&](int i) {
        float v = src0[i];
        for (int p = 1; p < n_part; ++p) v += src0[p * part_stride + i];
        return v;
    };
    const float2 *c = cs + t * half;
    const int q_dim = Hq * hd, kv_dim = Hkv * hd;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const T *bq = (const T *)ex.bq, *bk = (const T *)ex.bk, *bv = (const T *)ex.bv;
    // one warp per q or k head: lane owns pairs i = lane, lane + 32 (hd <= 128)
    // blockIdx.y spreads the heads of a row over several blocks (few rows: the resume call)
    for (int hh = warp + 4 * blockIdx.y; hh < Hq + Hkv; hh += 4 * gridDim.y) {
        const bool is_q = hh < Hq;
        if (is_q && !want_q) continue;
        const T *bias = is_q ? (bq ? bq + hh * hd : nullptr) : (bk ? bk + (hh - Hq) * hd : nullptr);
        const T *gain = (const T *)(is_q ? ex.qn : ex.kn);
        float x1[2], x2[2], ss = 0.f;
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            const int i = lane + 32 * e;
            x1[e] = x2[e] = 0.f;
            if (i < half) {
                x1[e] = src(hh * hd + i) + (bias ? to_f<T>(bias[i]) : 0.f);
                x2[e] = src(hh * hd + i + half) + (bias ? to_f<T>(bias[i + half]) : 0.f);
                ss += x1[e] * x1[e] + x2[e] * x2[e];
            }
        }
        if (gain) {
            ss = warp_sum(ss);
            const float inv = 1.0f / sqrtf(ss / (float)hd + ex.eps);
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int i = lane + 32 * e;
                if (i < half) {
                    x1[e] *= inv * to_f<T>(gain[i]);
                    x2[e] *= inv * to_f<T>(gain[i + half]);
                }
            }
        }
        T *dst = is_q ? q_out + t * q_dim + hh * hd : arena_k + (int64_t)slot[t] * kv_dim + (hh - Hq) * hd;
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            const int i = lane + 32 * e;
            if (i < half) {
                const float2 w = c[i];
                dst[i] = from_f<T>(x1[e] * w.x - x2[e] * w.y);
                dst[i + half] = from_f<T>(x2[e] * w.x + x1[e] * w.y);
            }
        }
    }
    if (kv_dim > 0) {
        T *vrow = arena_k + (int64_t)slot[t] * kv_dim + kv_stride;
        for (int idx = threadIdx.x + blockDim.x * blockIdx.y; idx < kv_dim; idx += blockDim.x * gridDim.y)
            vrow[idx] = from_f<T>(src(q_dim + kv_dim + idx) + (bv ? to_f<T>(bv[idx]) : 0.f));
    }
}

void launch_rope_scatter(bool fp32, const float *qkv, int ld, const float2 *cs, const ChunkMeta &cm,
                         const ModelDims &md, const ArenaView &av, int layer, bool want_q, void *q_out,
                         const QkvExtras &ex, cudaStream_t s, int n_part, int64_t part_stride, bool pdl) {
    if (cm.n == 0) return;
    // one block per row when there are rows enough to fill the GPU, else one block per four heads
    const dim3 grid(cm.n, cm.n >= 1024 ? 1 : (md.Hq + md.Hkv + 3) / 4);
    if (fp32) {
        float *ak = (float *)av.base + (int64_t)layer * av.layer_stride;
        launch_kernel(rope_scatter_kernel<float>, grid, dim3(128), 0, s, pdl, qkv, ld, n_part, part_stride, cs, cm.slot,
                      md.Hq, md.Hkv, md.hd, ak, av.kv_stride, want_q, (float *)q_out, ex);
    } else {
        __nv_bfloat16 *ak = (__nv_bfloat16 *)av.base + (int64_t)layer * av.layer_stride;
        launch_kernel(rope_scatter_kernel<__nv_bfloat16>, grid, dim3(128), 0, s, pdl, qkv, ld, n_part, part_stride, cs,
                      cm.slot, md.Hq, md.Hkv, md.hd, ak, av.kv_stride, want_q, (__nv_bfloat16 *)q_out, ex);
    }
}

// ---------------------------------------------------------------------------
// Causal attention over paged K/V, one warp per (query token, query head).
// Each lane owns hd/32 dims; keys are visited in order with a running softmax.
// ---------------------------------------------------------------------------
template <typename T, int EPL>
__global__ void __launch_bounds__(128) attn_simt_kernel(const T *__restrict__ q, const int32_t *__restrict__ pos,
                                                        const int32_t *__restrict__ trow,
                                                        const int32_t *__restrict__ tables, int max_blk, int Hq,
                                                        int Hkv, const T *__restrict__ arena_k, int64_t kv_stride,
                                                        int block_size, T *__restrict__ o) {
    constexpr int HD = EPL * 32;
    const int64_t t = blockIdx.x;
    const int hq = blockIdx.y * 4 + (threadIdx.x >> 5);
    if (hq >= Hq) return;
    const int lane = threadIdx.x & 31;
    const int hk = hq / (Hq / Hkv);
    const int q_dim = Hq * HD, kv_dim = Hkv * HD;
    const float scale = rsqrtf((float)HD);
    float qv[EPL], acc[EPL];
#pragma unroll
    for (int e = 0; e < EPL; ++e) {
        qv[e] = to_f<T>(q[t * q_dim + hq * HD + lane * EPL + e]) * scale;
        acc[e] = 0.f;
    }
    const int32_t *tab = tables + (int64_t)trow[t] * max_blk;
    const int p = pos[t];
    float m = -INFINITY, l = 0.f;
    for (int j = 0; j <= p; ++j) {
        const int64_t sl = (int64_t)tab[j / block_size] * block_size + (j % block_size);
        const T *kr = arena_k + sl * kv_dim + hk * HD + lane * EPL;
        const T *vr = kr + kv_stride;
        float s = 0.f;
#pragma unroll
        for (int e = 0; e < EPL; ++e) s = fmaf(qv[e], to_f<T>(kr[e]), s);
        s = warp_sum(s);
        const float mn = fmaxf(m, s);
        const float corr = expf(m - mn), pj = expf(s - mn);
        l = l * corr + pj;
#pragma unroll
        for (int e = 0; e < EPL; ++e) acc[e] = acc[e] * corr + pj * to_f<T>(vr[e]);
        m = mn;
    }
    const float inv = 1.0f / l;
#pragma unroll
    for (int e = 0; e < EPL; ++e) o[t * q_dim + hq * HD + lane * EPL + e] = from_f<T>(acc[e] * inv);
}

void launch_attn_simt(bool fp32, const void *q, const ChunkMeta &cm, const int32_t *tables, int max_blk,
                      const ModelDims &md, const ArenaView &av, int layer, void *o, cudaStream_t s) {
    if (cm.n == 0) return;
    dim3 grid(cm.n, (md.Hq + 3) / 4);
#define KVR_ATTN(T, EPL)                                                                                      \
    attn_simt_kernel<T, EPL><<<grid, 128, 0, s>>>((const T *)q, cm.pos, cm.trow, tables, max_blk, md.Hq,      \
                                                  md.Hkv, (const T *)av.base + (int64_t)layer * av.layer_stride, \
                                                  av.kv_stride, av.block_size, (T *)o)
    if (fp32) {
        if (md.hd == 64) KVR_ATTN(float, 2); else KVR_ATTN(float, 4);
    } else {
        if (md.hd == 64) KVR_ATTN(__nv_bfloat16, 2); else KVR_ATTN(__nv_bfloat16, 4);
    }
#undef KVR_ATTN
}

// ---------------------------------------------------------------------------
// Read-back gather: arena rows of one request and layer -> dense [n, Hkv*hd].
// 16-byte copies; row bytes are a multiple of 16 (host checks).
// ---------------------------------------------------------------------------
__global__ void readback_kernel(const uint4 *__restrict__ arena_k, int64_t kv_stride_v, int row_v,
                                const int32_t *__restrict__ table, int block_size, int n,
                                uint4 *__restrict__ k_out, uint4 *__restrict__ v_out) {
    const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (int64_t)n * row_v) return;
    const int t = (int)(idx / row_v), c = (int)(idx % row_v);
    const int64_t sl = (int64_t)table[t / block_size] * block_size + (t % block_size);
    const uint4 *src = arena_k + sl * row_v + c;
    k_out[idx] = src[0];
    v_out[idx] = src[kv_stride_v];
}

void launch_readback(bool fp32, const ArenaView &av, int layer, const int32_t *table_dev, int n, void *k_out,
                     void *v_out, cudaStream_t s) {
    if (n == 0) return;
    const int es = fp32 ? 4 : 2;
    const int row_v = av.row * es / 16;
    const int64_t kvs_v = av.kv_stride * es / 16;
    const uint4 *base = (const uint4 *)((const char *)av.base + (int64_t)layer * av.layer_stride * es);
    const int64_t total = (int64_t)n * row_v;
    readback_kernel<<<(unsigned)((total + 255) / 256), 256, 0, s>>>(base, kvs_v, row_v, table_dev, av.block_size, n,
                                                                    (uint4 *)k_out, (uint4 *)v_out);
}

// ---------------------------------------------------------------------------
// Copies the residual rows of the tokens that end their request into the
// per-request buffer used to resume decoding: h_last[pair.y] = h[pair.x].
// ---------------------------------------------------------------------------
__global__ void gather_rows_kernel(const float *__restrict__ h, int d, const int2 *__restrict__ pairs,
                                   float *__restrict__ h_last) {
    const int2 pr = pairs[blockIdx.x];
    const float4 *src = reinterpret_cast<const float4 *>(h + (int64_t)pr.x * d);
    float4 *dst = reinterpret_cast<float4 *>(h_last + (int64_t)pr.y * d);
    for (int i = threadIdx.x; i < d / 4; i += blockDim.x) dst[i] = src[i];
}

void launch_gather_rows(const float *h, int d, const int2 *pairs, int n_pairs, float *h_last, cudaStream_t s) {
    if (n_pairs > 0) gather_rows_kernel<<<n_pairs, 128, 0, s>>>(h, d, pairs, h_last);
}

}  // namespace kvr
