// Persistent warp-specialised bf16 GEMM on tcgen05: C[M,N] = A[M,K] W[N,K]^T,
// operands staged by TMA (128-byte swizzle), accumulators in TMEM (two buffers,
// so one tile's epilogue overlaps the next tile's MMAs), fused epilogues:
//   TC_STORE_F32 / TC_RESID  fp32 store / fp32 residual add
//   TC_SWIGLU                gate and up rows share a tile: out = silu(g) * u (bf16)
//   TC_QKV                   RoPE on q/k, q -> workspace, k/v -> paged arena rows
// Tile 128 x 256 x 64, 4-stage ring; warp 0 = TMA producer, warp 1 = MMA issuer,
// warps 2..5 = epilogue (each owns the 32 TMEM lanes its warp id selects).
// Two tilings share the epilogues: gemm_tc_kernel (one CTA per 128 x 256 tile) and
// gemm_tc2_kernel (a CTA pair per 256 x 256 tile, tcgen05 cta_group::2; the default).
#include "kvr_internal.h"
#include "kvr_ptx.cuh"

namespace kvr {

namespace {

constexpr int BM = 128, BN = 256, BK = 64, STAGES = 4, UMMA_K = 16;
constexpr int A_BYTES = BM * BK * 2;          // 16 KB
constexpr int BH_BYTES = 128 * BK * 2;        // one 128-row half of B
constexpr int STAGE_BYTES = A_BYTES + 2 * BH_BYTES;
constexpr int TMEM_COLS = 512;
constexpr int STG_WARP_BYTES = 2 * 4096;     // per epilogue warp: two 32-row x 128-byte staging tiles
constexpr int STG_BYTES = 4 * STG_WARP_BYTES;
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + STG_BYTES + 1024 /*align slack*/ + 256 /*barriers*/;
constexpr int N_THREADS = 192;

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;

struct TileCoord { int m, n; };

__device__ __forceinline__ TileCoord tile_coord(int t, int num_m, int num_n, int gn) {
    const int per_panel = gn * num_m;
    const int panel = t / per_panel;
    const int within = t - panel * per_panel;
    const int width = min(gn, num_n - panel * gn);
    TileCoord c;
    c.m = within / width;
    c.n = panel * gn + (within - c.m * width);
    return c;
}

// Which weight operand and which of its rows feed half `hf` of N tile `nt`.
__device__ __forceinline__ void half_source(const TcGemmEpilogue &ep, int nt, int hf, int &op, int &row) {
    if (ep.mode == TC_SWIGLU) {
        op = hf;
        row = nt * 128;
    } else if (ep.mode == TC_QKV) {
        int col = (nt * 2 + hf) * 128;
        op = 0;
        row = ep.b_rows[0];  // first row past the operand: the load is zero-filled
        if (col < ep.b_rows[0]) { op = 0; row = col; return; }
        col -= ep.b_rows[0];
        if (col < ep.b_rows[1]) { op = 1; row = col; return; }
        col -= ep.b_rows[1];
        if (col < ep.b_rows[2]) { op = 2; row = col; return; }
    } else {
        op = 0;
        row = nt * BN + hf * 128;
    }
}

__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
    __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t *>(&h);
}

__device__ __forceinline__ void epilogue_plain(const TcGemmEpilogue &ep, uint32_t tacc, int row, int n0) {
#pragma unroll 1
    for (int c = 0; c < BN; c += 32) {
        uint32_t r[32];
        ptx::tmem_ld32(tacc + c, r);
        ptx::tmem_ld_wait();
        if (row >= ep.M) continue;
        float *dst = ep.c_f32 + (int64_t)row * ep.ldc + n0 + c;
        const int ncol = ep.N - (n0 + c);
        if (ncol >= 32 && (ep.ldc & 3) == 0) {
#pragma unroll
            for (int j = 0; j < 32; j += 4) {
                float4 v = make_float4(__uint_as_float(r[j]), __uint_as_float(r[j + 1]), __uint_as_float(r[j + 2]),
                                       __uint_as_float(r[j + 3]));
                if (ep.mode == TC_RESID) {
                    const float4 o = *reinterpret_cast<const float4 *>(dst + j);
                    v.x += o.x; v.y += o.y; v.z += o.z; v.w += o.w;
                }
                *reinterpret_cast<float4 *>(dst + j) = v;
            }
        } else {
#pragma unroll
            for (int j = 0; j < 32; ++j)
                if (j < ncol) {
                    float v = __uint_as_float(r[j]);
                    if (ep.mode == TC_RESID) v += dst[j];
                    dst[j] = v;
                }
        }
    }
}

// Residual add through the copy engine: the accumulator chunk (32 rows x 32 fp32 columns per
// warp) is staged in shared memory in the 128-byte-swizzle layout and added to h by a TMA
// reduce.  Every element of h is touched by exactly one such add per launch, so the result
// does not depend on any ordering.  Rows and columns past the matrix are clipped by the map.
__device__ __forceinline__ void epilogue_resid_tma(const TcGemmEpilogue &ep, const CUtensorMap *tmH, uint32_t tacc,
                                                   uint32_t stg, int lane, int row0, int n0) {
#pragma unroll 1
    for (int c = 0; c < BN; c += 32) {
        const uint32_t buf = stg + ((c >> 5) & 1) * 4096;
        if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");   // buffer free again
        __syncwarp();
        uint32_t r[32];
        ptx::tmem_ld32(tacc + c, r);
        ptx::tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const uint32_t dst = buf + lane * 128 + ((j ^ (lane & 7)) << 4);
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(r[4 * j]), "r"(r[4 * j + 1]),
                         "r"(r[4 * j + 2]), "r"(r[4 * j + 3]) : "memory");
        }
        ptx::fence_proxy_async();
        __syncwarp();
        if (lane == 0 && n0 + c < ep.N && row0 < ep.M) {
            asm volatile(
                "cp.reduce.async.bulk.tensor.2d.global.shared::cta.add.tile.bulk_group [%0, {%1, %2}], [%3];"
                ::"l"(tmH), "r"(n0 + c), "r"(row0), "r"(buf) : "memory");
            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        }
    }
}

__device__ __forceinline__ void epilogue_swiglu(const TcGemmEpilogue &ep, uint32_t tacc, int row, int nt) {
    const int F = ep.N >> 1;
#pragma unroll 1
    for (int c = 0; c < 128; c += 16) {
        uint32_t g[16], u[16];
        ptx::tmem_ld16(tacc + c, g);
        ptx::tmem_ld16(tacc + 128 + c, u);
        ptx::tmem_ld_wait();
        const int col = nt * 128 + c;
        if (row >= ep.M || col >= F) continue;
        uint32_t o[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const float g0 = __uint_as_float(g[2 * j]), g1 = __uint_as_float(g[2 * j + 1]);
            const float s0 = g0 / (1.0f + __expf(-g0)), s1 = g1 / (1.0f + __expf(-g1));
            o[j] = pack_bf16(s0 * __uint_as_float(u[2 * j]), s1 * __uint_as_float(u[2 * j + 1]));
        }
        __nv_bfloat16 *dst = ep.out_bf16 + (int64_t)row * ep.ld_out + col;
        // streaming stores: m is far larger than L2 and must not push the A operand out of it
        if (col + 16 <= F) {
            __stcs(reinterpret_cast<uint4 *>(dst), make_uint4(o[0], o[1], o[2], o[3]));
            __stcs(reinterpret_cast<uint4 *>(dst + 8), make_uint4(o[4], o[5], o[6], o[7]));
        } else {  // F is a multiple of 8
            __stcs(reinterpret_cast<uint4 *>(dst), make_uint4(o[0], o[1], o[2], o[3]));
        }
    }
}

// The same with the optional projection terms: bias on q/k/v, per-head RMSNorm of q and k
// (sum of squares over the head's columns in a first pass over TMEM) before the rotation.
__device__ __forceinline__ void epilogue_qkv_ext(const TcGemmEpilogue &ep, uint32_t tacc, int row, int nt) {
    const int hd = ep.head_dim, half = hd >> 1;
    const bool live = row < ep.M;
    const int64_t slot = live ? ep.slot[row] : 0;
    const float2 *cs = ep.rope_cs + (int64_t)(live ? row : 0) * half;
#pragma unroll 1
    for (int hf = 0; hf < 2; ++hf) {
        const int col0 = (nt * 2 + hf) * 128;
        __nv_bfloat16 *dst;
        const __nv_bfloat16 *bias, *gain = nullptr;
        bool rotate = true;
        if (col0 < ep.n_q_cols) {
            dst = ep.q_out + (int64_t)row * ep.n_q_cols + col0;
            bias = ep.bias_q ? ep.bias_q + col0 : nullptr;
            gain = ep.gain_q;
        } else if (col0 < ep.n_q_cols + ep.n_kv_cols) {
            dst = ep.arena_k + slot * ep.n_kv_cols + (col0 - ep.n_q_cols);
            bias = ep.bias_k ? ep.bias_k + (col0 - ep.n_q_cols) : nullptr;
            gain = ep.gain_k;
        } else if (col0 < ep.n_q_cols + 2 * ep.n_kv_cols) {
            dst = ep.arena_k + ep.kv_stride + slot * ep.n_kv_cols + (col0 - ep.n_q_cols - ep.n_kv_cols);
            bias = ep.bias_v ? ep.bias_v + (col0 - ep.n_q_cols - ep.n_kv_cols) : nullptr;
            rotate = false;
        } else {
            continue;  // uniform over the CTA
        }
        if (!rotate) {
#pragma unroll 1
            for (int c = 0; c < 128; c += 16) {
                uint32_t r[16];
                ptx::tmem_ld16(tacc + hf * 128 + c, r);
                ptx::tmem_ld_wait();
                if (!live) continue;
                uint32_t y[8];
#pragma unroll
                for (int j = 0; j < 16; j += 2) {
                    const float b0 = bias ? __bfloat162float(bias[c + j]) : 0.f;
                    const float b1 = bias ? __bfloat162float(bias[c + j + 1]) : 0.f;
                    y[j >> 1] = pack_bf16(__uint_as_float(r[j]) + b0, __uint_as_float(r[j + 1]) + b1);
                }
                *reinterpret_cast<uint4 *>(dst + c) = make_uint4(y[0], y[1], y[2], y[3]);
                *reinterpret_cast<uint4 *>(dst + c + 8) = make_uint4(y[4], y[5], y[6], y[7]);
            }
            continue;
        }
#pragma unroll 1
        for (int hs = 0; hs < 128; hs += hd) {
            float inv = 1.f;
            if (gain) {
                float ss = 0.f;
#pragma unroll 1
                for (int c = 0; c < hd; c += 16) {
                    uint32_t r[16];
                    ptx::tmem_ld16(tacc + hf * 128 + hs + c, r);
                    ptx::tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const float x = __uint_as_float(r[j]) + (bias ? __bfloat162float(bias[hs + c + j]) : 0.f);
                        ss = fmaf(x, x, ss);
                    }
                }
                inv = rsqrtf(ss / (float)hd + ep.qk_eps);
            }
#pragma unroll 1
            for (int i0 = 0; i0 < half; i0 += 16) {
                uint32_t x1[16], x2[16];
                ptx::tmem_ld16(tacc + hf * 128 + hs + i0, x1);
                ptx::tmem_ld16(tacc + hf * 128 + hs + half + i0, x2);
                ptx::tmem_ld_wait();
                if (!live) continue;
                uint32_t y1[8], y2[8];
                float a[2], b[2];
#pragma unroll
                for (int j = 0; j < 16; j += 2) {
                    const float4 w = *reinterpret_cast<const float4 *>(cs + i0 + j);  // (c0, s0, c1, s1)
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        const int i = hs + i0 + j + e;
                        a[e] = __uint_as_float(x1[j + e]) + (bias ? __bfloat162float(bias[i]) : 0.f);
                        b[e] = __uint_as_float(x2[j + e]) + (bias ? __bfloat162float(bias[i + half]) : 0.f);
                        if (gain) {
                            a[e] *= inv * __bfloat162float(gain[i0 + j + e]);
                            b[e] *= inv * __bfloat162float(gain[half + i0 + j + e]);
                        }
                    }
                    y1[j >> 1] = pack_bf16(a[0] * w.x - b[0] * w.y, a[1] * w.z - b[1] * w.w);
                    y2[j >> 1] = pack_bf16(b[0] * w.x + a[0] * w.y, b[1] * w.z + a[1] * w.w);
                }
                __nv_bfloat16 *d1 = dst + hs + i0, *d2 = dst + hs + half + i0;
                *reinterpret_cast<uint4 *>(d1) = make_uint4(y1[0], y1[1], y1[2], y1[3]);
                *reinterpret_cast<uint4 *>(d1 + 8) = make_uint4(y1[4], y1[5], y1[6], y1[7]);
                *reinterpret_cast<uint4 *>(d2) = make_uint4(y2[0], y2[1], y2[2], y2[3]);
                *reinterpret_cast<uint4 *>(d2 + 8) = make_uint4(y2[4], y2[5], y2[6], y2[7]);
            }
        }
    }
}

__device__ __forceinline__ void epilogue_qkv(const TcGemmEpilogue &ep, uint32_t tacc, int row, int nt) {
    const int hd = ep.head_dim, half = hd >> 1;
    const bool live = row < ep.M;
    const int64_t slot = live ? ep.slot[row] : 0;
    const float2 *cs = ep.rope_cs + (int64_t)(live ? row : 0) * half;
#pragma unroll 1
    for (int hf = 0; hf < 2; ++hf) {
        int col0 = (nt * 2 + hf) * 128;
        int kind;  // 0 q, 1 k, 2 v, 3 nothing
        __nv_bfloat16 *dst = nullptr;
        if (col0 < ep.n_q_cols) {
            kind = 0;
            dst = ep.q_out + (int64_t)row * ep.n_q_cols + col0;
        } else if (col0 < ep.n_q_cols + ep.n_kv_cols) {
            kind = 1;
            dst = ep.arena_k + slot * ep.n_kv_cols + (col0 - ep.n_q_cols);
        } else if (col0 < ep.n_q_cols + 2 * ep.n_kv_cols) {
            kind = 2;
            dst = ep.arena_k + ep.kv_stride + slot * ep.n_kv_cols + (col0 - ep.n_q_cols - ep.n_kv_cols);
        } else {
            kind = 3;
        }
        if (kind == 3) continue;  // uniform over the CTA
        if (kind == 2) {
#pragma unroll 1
            for (int c = 0; c < 128; c += 32) {
                uint32_t r[32];
                ptx::tmem_ld32(tacc + hf * 128 + c, r);
                ptx::tmem_ld_wait();
                if (!live) continue;
#pragma unroll
                for (int j = 0; j < 32; j += 8)
                    *reinterpret_cast<uint4 *>(dst + c + j) = make_uint4(
                        pack_bf16(__uint_as_float(r[j]), __uint_as_float(r[j + 1])),
                        pack_bf16(__uint_as_float(r[j + 2]), __uint_as_float(r[j + 3])),
                        pack_bf16(__uint_as_float(r[j + 4]), __uint_as_float(r[j + 5])),
                        pack_bf16(__uint_as_float(r[j + 6]), __uint_as_float(r[j + 7])));
            }
            continue;
        }
        // rotate-half RoPE: element i pairs with i + hd/2 inside each head
#pragma unroll 1
        for (int hs = 0; hs < 128; hs += hd) {
#pragma unroll 1
            for (int i0 = 0; i0 < half; i0 += 16) {
                uint32_t x1[16], x2[16];
                ptx::tmem_ld16(tacc + hf * 128 + hs + i0, x1);
                ptx::tmem_ld16(tacc + hf * 128 + hs + half + i0, x2);
                ptx::tmem_ld_wait();
                if (!live) continue;
                uint32_t y1[8], y2[8];
#pragma unroll
                for (int j = 0; j < 16; j += 2) {
                    const float4 w = *reinterpret_cast<const float4 *>(cs + i0 + j);  // (c0, s0, c1, s1)
                    const float a0 = __uint_as_float(x1[j]), b0 = __uint_as_float(x2[j]);
                    const float a1 = __uint_as_float(x1[j + 1]), b1 = __uint_as_float(x2[j + 1]);
                    y1[j >> 1] = pack_bf16(a0 * w.x - b0 * w.y, a1 * w.z - b1 * w.w);
                    y2[j >> 1] = pack_bf16(b0 * w.x + a0 * w.y, b1 * w.z + a1 * w.w);
                }
                __nv_bfloat16 *d1 = dst + hs + i0, *d2 = dst + hs + half + i0;
                *reinterpret_cast<uint4 *>(d1) = make_uint4(y1[0], y1[1], y1[2], y1[3]);
                *reinterpret_cast<uint4 *>(d1 + 8) = make_uint4(y1[4], y1[5], y1[6], y1[7]);
                *reinterpret_cast<uint4 *>(d2) = make_uint4(y2[0], y2[1], y2[2], y2[3]);
                *reinterpret_cast<uint4 *>(d2 + 8) = make_uint4(y2[4], y2[5], y2[6], y2[7]);
            }
        }
    }
}

// EXT: the QKV epilogue applies the optional bias / per-head norm terms.
template <bool EXT>
__global__ void __launch_bounds__(N_THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB0,
               const __grid_constant__ CUtensorMap tmB1, const __grid_constant__ CUtensorMap tmB2,
               const __grid_constant__ CUtensorMap tmH, const TcGemmEpilogue ep, int num_m, int num_n, int gn, int *status) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = ptx::smem_u32(smem_raw);
    const uint32_t tiles = (raw + 1023u) & ~1023u;  // stage s at tiles + s * STAGE_BYTES
    const uint32_t stg0 = tiles + STAGES * STAGE_BYTES;   // epilogue staging, 1024-byte aligned
    const uint32_t bars = stg0 + STG_BYTES;
    // barrier addresses: full[s], empty[s], tmem_full[2], tmem_empty[2]
    const uint32_t full0 = bars, empty0 = bars + 8 * STAGES, tfull0 = bars + 16 * STAGES,
                   tempty0 = bars + 16 * STAGES + 16;
    __shared__ uint32_t tmem_base_sh;
    __shared__ int abort_sh;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        abort_sh = 0;
        for (int s = 0; s < STAGES; ++s) {
            ptx::mbar_init(full0 + 8 * s, 1);
            ptx::mbar_init(empty0 + 8 * s, 1);
        }
        for (int a = 0; a < 2; ++a) {
            ptx::mbar_init(tfull0 + 8 * a, 1);
            ptx::mbar_init(tempty0 + 8 * a, 4);
        }
        ptx::fence_mbar_init();
        ptx::prefetch_tmap(&tmA);
        ptx::prefetch_tmap(&tmB0);
    }
    if (warp == 1) {
        ptx::tmem_alloc(ptx::smem_u32(&tmem_base_sh), TMEM_COLS);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = tmem_base_sh;
    volatile int *abort_flag = &abort_sh;

    const int total_tiles = num_m * num_n;
    const int num_k = (ep.K + BK - 1) / BK;

    if (warp == 0) {
        if (lane == 0 && !ptx::loads_muted(status)) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
                const TileCoord tc = tile_coord(t, num_m, num_n, gn);
                int op0, row0, op1, row1;
                half_source(ep, tc.n, 0, op0, row0);
                half_source(ep, tc.n, 1, op1, row1);
                const CUtensorMap *m0 = op0 == 0 ? &tmB0 : (op0 == 1 ? &tmB1 : &tmB2);
                const CUtensorMap *m1 = op1 == 0 ? &tmB0 : (op1 == 1 ? &tmB1 : &tmB2);
                for (int kb = 0; kb < num_k; ++kb) {
                    if (!ptx::mbar_wait(empty0 + 8 * stage, phase ^ 1u, status, abort_flag)) { ok = false; break; }
                    const uint32_t fb = full0 + 8 * stage;
                    const uint32_t sa = tiles + stage * STAGE_BYTES;
                    ptx::mbar_expect_tx(fb, STAGE_BYTES);
                    ptx::tma_load_2d(sa, &tmA, kb * BK, tc.m * BM, fb);
                    ptx::tma_load_2d(sa + A_BYTES, m0, kb * BK, row0, fb);
                    ptx::tma_load_2d(sa + A_BYTES + BH_BYTES, m1, kb * BK, row1, fb);
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t IDESC = ptx::idesc_bf16(BM, BN);
            int stage = 0;
            uint32_t phase = 0, acc_phase = 0;
            int acc = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
                if (!ptx::mbar_wait(tempty0 + 8 * acc, acc_phase ^ 1u, status, abort_flag)) { ok = false; break; }
                ptx::tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * BN;
                for (int kb = 0; kb < num_k; ++kb) {
                    if (!ptx::mbar_wait(full0 + 8 * stage, phase, status, abort_flag)) { ok = false; break; }
                    ptx::tc_fence_after();
                    const uint32_t sa = tiles + stage * STAGE_BYTES;
                    const uint64_t da = ptx::smem_desc_sw128(sa);
                    const uint64_t db = ptx::smem_desc_sw128(sa + A_BYTES);
#pragma unroll
                    for (int kk = 0; kk < BK / UMMA_K; ++kk) {
                        // +32 bytes along K inside the swizzled row = +2 in the address field
                        ptx::mma_bf16_ss(d_tmem, da + 2 * kk, db + 2 * kk, IDESC, (kb | kk) != 0);
                    }
                    ptx::mma_commit(empty0 + 8 * stage);
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                ptx::mma_commit(tfull0 + 8 * acc);
                if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
            }
        }
    } else {
        const int quarter = warp & 3;  // TMEM lanes this warp may read
        uint32_t acc_phase = 0;
        int acc = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
            const TileCoord tc = tile_coord(t, num_m, num_n, gn);
            if (!ptx::mbar_wait(tfull0 + 8 * acc, acc_phase, status, abort_flag)) { ok = false; break; }
            ptx::tc_fence_after();
            const uint32_t tacc = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * BN;
            const int row = tc.m * BM + quarter * 32 + lane;
            if (ep.mode == TC_QKV) {
                if (EXT) epilogue_qkv_ext(ep, tacc, row, tc.n);
                else epilogue_qkv(ep, tacc, row, tc.n);
            }
            else if (ep.mode == TC_SWIGLU) epilogue_swiglu(ep, tacc, row, tc.n);
            else if (ep.mode == TC_RESID && ep.resid_tma)
                epilogue_resid_tma(ep, &tmH, tacc, stg0 + (warp - 2) * STG_WARP_BYTES, lane,
                                   tc.m * BM + quarter * 32, tc.n * BN);
            else epilogue_plain(ep, tacc, row, tc.n * BN);
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(tempty0 + 8 * acc);
            if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
        }
        if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");   // reduces have landed
    }
    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

// ---------------------------------------------------------------------------
// The same GEMM on CTA pairs (cluster of two, tcgen05 cta_group::2): one 256 x 256 output
// tile per pair.  Each CTA stages its own 128 rows of A and one 128-row half of the weight
// tile (32 KB per k-block instead of 48, so six stages fit and a third less data crosses from
// L2 to shared memory per flop); the leader CTA's MMA warp issues one M = 256 instruction for
// both, each CTA's TMEM receives its 128 rows of the accumulator and its own epilogue warps
// drain them.  Barriers: every TMA load of either CTA counts on the leader's full[s]; the
// leader's commits arrive on empty[s] and tmem_full[a] of both CTAs; the epilogue warps of
// both CTAs arrive on the leader's tmem_empty[a].
// ---------------------------------------------------------------------------
constexpr int STAGES2 = 6;
constexpr int STAGE2_BYTES = A_BYTES + BH_BYTES;   // 32 KB
constexpr int SMEM2_BYTES = STAGES2 * STAGE2_BYTES + STG_BYTES + 1024 + 256;

template <bool EXT>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(N_THREADS, 1)
gemm_tc2_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB0,
                const __grid_constant__ CUtensorMap tmB1, const __grid_constant__ CUtensorMap tmB2,
                const __grid_constant__ CUtensorMap tmH, const TcGemmEpilogue ep, int num_m, int num_n, int gn,
                int *status) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = ptx::smem_u32(smem_raw);
    const uint32_t tiles = (raw + 1023u) & ~1023u;
    const uint32_t stg0 = tiles + STAGES2 * STAGE2_BYTES;
    const uint32_t bars = stg0 + STG_BYTES;
    const uint32_t full0 = bars, empty0 = bars + 8 * STAGES2, tfull0 = bars + 16 * STAGES2,
                   tempty0 = bars + 16 * STAGES2 + 16;
    __shared__ uint32_t tmem_base_sh;
    __shared__ int abort_sh;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = ptx::cluster_ctarank();
    const bool leader = rank == 0;
    const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
    if (threadIdx.x == 0) {
        abort_sh = 0;
        for (int s = 0; s < STAGES2; ++s) {
            ptx::mbar_init(full0 + 8 * s, 1);
            ptx::mbar_init(empty0 + 8 * s, 1);
        }
        for (int a = 0; a < 2; ++a) {
            ptx::mbar_init(tfull0 + 8 * a, 1);
            ptx::mbar_init(tempty0 + 8 * a, 8);
        }
        ptx::fence_mbar_init();
        ptx::prefetch_tmap(&tmA);
        ptx::prefetch_tmap(&tmB0);
    }
    if (warp == 1) {
        ptx::tmem_alloc_pair(ptx::smem_u32(&tmem_base_sh), TMEM_COLS);
        ptx::tmem_relinquish_pair();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::cluster_sync();   // the peer's barriers are initialised before anything signals them
    ptx::tc_fence_after();
    const uint32_t tmem_base = tmem_base_sh;
    volatile int *abort_flag = &abort_sh;

    const int total_tiles = num_m * num_n;
    const int num_k = (ep.K + BK - 1) / BK;

    if (warp == 0) {
        if (lane == 0 && !ptx::loads_muted(status)) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int t = pair; t < total_tiles && ok; t += n_pairs) {
                const TileCoord tc = tile_coord(t, num_m, num_n, gn);
                int op, brow;
                half_source(ep, tc.n, (int)rank, op, brow);
                const CUtensorMap *mb = op == 0 ? &tmB0 : (op == 1 ? &tmB1 : &tmB2);
                const int arow = tc.m * 256 + (int)rank * 128;
                for (int kb = 0; kb < num_k; ++kb) {
                    if (!ptx::mbar_wait(empty0 + 8 * stage, phase ^ 1u, status, abort_flag)) { ok = false; break; }
                    const uint32_t fb = ptx::map_to_cta(full0 + 8 * stage, 0);
                    const uint32_t sa = tiles + stage * STAGE2_BYTES;
                    if (leader) ptx::mbar_expect_tx(full0 + 8 * stage, 2 * STAGE2_BYTES);
                    ptx::tma_load_2d_pair(sa, &tmA, kb * BK, arow, fb);
                    ptx::tma_load_2d_pair(sa + A_BYTES, mb, kb * BK, brow, fb);
                    if (++stage == STAGES2) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && leader) {
            constexpr uint32_t IDESC = ptx::idesc_bf16(256, BN);
            int stage = 0;
            uint32_t phase = 0, acc_phase = 0;
            int acc = 0;
            bool ok = true;
            for (int t = pair; t < total_tiles && ok; t += n_pairs) {
                if (!ptx::mbar_wait(tempty0 + 8 * acc, acc_phase ^ 1u, status, abort_flag)) { ok = false; break; }
                ptx::tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * BN;
                for (int kb = 0; kb < num_k; ++kb) {
                    if (!ptx::mbar_wait(full0 + 8 * stage, phase, status, abort_flag)) { ok = false; break; }
                    ptx::tc_fence_after();
                    const uint32_t sa = tiles + stage * STAGE2_BYTES;
                    const uint64_t da = ptx::smem_desc_sw128(sa);
                    const uint64_t db = ptx::smem_desc_sw128(sa + A_BYTES);
#pragma unroll
                    for (int kk = 0; kk < BK / UMMA_K; ++kk)
                        ptx::mma_bf16_ss_pair(d_tmem, da + 2 * kk, db + 2 * kk, IDESC, (kb | kk) != 0);
                    ptx::mma_commit_pair(empty0 + 8 * stage, 3);
                    if (++stage == STAGES2) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                ptx::mma_commit_pair(tfull0 + 8 * acc, 3);
                if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
            }
        }
    } else {
        const int quarter = warp & 3;
        uint32_t acc_phase = 0;
        int acc = 0;
        bool ok = true;
        for (int t = pair; t < total_tiles && ok; t += n_pairs) {
            const TileCoord tc = tile_coord(t, num_m, num_n, gn);
            if (!ptx::mbar_wait(tfull0 + 8 * acc, acc_phase, status, abort_flag)) { ok = false; break; }
            ptx::tc_fence_after();
            const uint32_t tacc = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * BN;
            const int row0 = tc.m * 256 + (int)rank * 128 + quarter * 32;
            const int row = row0 + lane;
            if (ep.mode == TC_QKV) {
                if (EXT) epilogue_qkv_ext(ep, tacc, row, tc.n);
                else epilogue_qkv(ep, tacc, row, tc.n);
            }
            else if (ep.mode == TC_SWIGLU) epilogue_swiglu(ep, tacc, row, tc.n);
            else if (ep.mode == TC_RESID && ep.resid_tma)
                epilogue_resid_tma(ep, &tmH, tacc, stg0 + (warp - 2) * STG_WARP_BYTES, lane, row0, tc.n * BN);
            else epilogue_plain(ep, tacc, row, tc.n * BN);
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive_cluster(ptx::map_to_cta(tempty0 + 8 * acc, 0));
            if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
        }
        if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");   // reduces have landed
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::cluster_sync();   // neither CTA's shared memory or TMEM is released while the other may use it
    if (warp == 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc_pair(tmem_base, TMEM_COLS);
    }
}

}  // namespace

int tc_gemm_init(int device) {
    (void)device;
    if (!g_encode) {
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
            qres != cudaDriverEntryPointSuccess || !fn)
            return KVR_ERR_CUDA;
        g_encode = (EncodeTiledFn)fn;
    }
    if (cudaFuncSetAttribute(gemm_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES) !=
            cudaSuccess ||
        cudaFuncSetAttribute(gemm_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES) !=
            cudaSuccess ||
        cudaFuncSetAttribute(gemm_tc2_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM2_BYTES) !=
            cudaSuccess ||
        cudaFuncSetAttribute(gemm_tc2_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM2_BYTES) !=
            cudaSuccess)
        return KVR_ERR_CUDA;
    return KVR_OK;
}

// Row-major [rows, cols] bf16 matrix; box = box_rows x box_cols with the
// 128-byte swizzle (box_cols * 2 must be 128).
int tc_make_tmap_2d(CUtensorMap *out, const void *base, int64_t rows, int64_t cols, int box_rows, int box_cols) {
    if (!g_encode) return KVR_ERR_UNSUPPORTED;
    if (((uintptr_t)base) % 16 || (cols * 2) % 16) return KVR_ERR_UNSUPPORTED;
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
    cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = g_encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box,
                          estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? KVR_OK : KVR_ERR_CUDA;
}

// Paged K/V planes seen as [rows, cols] bf16 (one row = one slot, all kv heads), cut for
// block gathers: dimensions (64 dims, 8 slots, 64-dim column group, 8-slot group), so that
// one box = `halves` column groups x 16 slots lands as [8-slot group][half][8 slots][128 B],
// the 128-byte-swizzled layout both MMA operand kinds read.
int tc_make_tmap_kv(CUtensorMap *out, const void *base, int64_t rows, int64_t cols, int halves) {
    if (!g_encode) return KVR_ERR_UNSUPPORTED;
    if (((uintptr_t)base) % 16 || cols % 64 || rows % 8) return KVR_ERR_UNSUPPORTED;
    cuuint64_t dims[4] = {64, 8, (cuuint64_t)(cols / 64), (cuuint64_t)(rows / 8)};
    cuuint64_t strides[3] = {(cuuint64_t)cols * 2, 128, (cuuint64_t)cols * 16};
    cuuint32_t box[4] = {64, 8, (cuuint32_t)halves, 2};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = g_encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(base), dims, strides, box,
                          estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? KVR_OK : KVR_ERR_CUDA;
}

// Row-major [rows, cols] fp32 matrix; box = 32 x 32 with the 128-byte swizzle (reduce/store target).
int tc_make_tmap_f32(CUtensorMap *out, const void *base, int64_t rows, int64_t cols) {
    if (!g_encode) return KVR_ERR_UNSUPPORTED;
    if (((uintptr_t)base) % 16 || (cols * 4) % 16) return KVR_ERR_UNSUPPORTED;
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)cols * 4};
    cuuint32_t box[2] = {32, 32};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = g_encode(out, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void *>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? KVR_OK : KVR_ERR_CUDA;
}

int launch_gemm_tc(const CUtensorMap &tmA, const CUtensorMap *tmB, const TcGemmEpilogue &ep_in, int *d_status,
                   int n_sms, cudaStream_t s, const CUtensorMap *tmH, bool pair) {
    TcGemmEpilogue ep = ep_in;
    ep.resid_tma = (tmH != nullptr && ep.mode == TC_RESID) ? 1 : 0;
    if (ep.M <= 0) return KVR_OK;
    int n_tiles_n;
    if (ep.mode == TC_SWIGLU) n_tiles_n = (ep.N / 2 + 127) / 128;
    else n_tiles_n = (ep.N + BN - 1) / BN;
    // tiles are rasterised in panels of PANEL_N column tiles: a wave of CTAs shares a few row tiles of A
    // and the panel's weight rows through L2 (8 ... 24 measured on the 7B workload: 16 best by 1 %)
    constexpr int PANEL_N = 16;
    const int gn = n_tiles_n < PANEL_N ? n_tiles_n : PANEL_N;
    const bool ext = ep.mode == TC_QKV && (ep.bias_q || ep.bias_k || ep.bias_v || ep.gain_q || ep.gain_k);
    const CUtensorMap &th = tmH ? *tmH : tmA;
    if (pair) {
        const int num_m = (ep.M + 255) / 256;
        const int total = num_m * n_tiles_n;
        const int n_pairs = total < n_sms / 2 ? total : n_sms / 2;
        if (n_pairs < 1) return KVR_ERR_UNSUPPORTED;
        if (ext)
            gemm_tc2_kernel<true><<<2 * n_pairs, N_THREADS, SMEM2_BYTES, s>>>(tmA, tmB[0], tmB[1], tmB[2], th, ep, num_m,
                                                                             n_tiles_n, gn, d_status);
        else
            gemm_tc2_kernel<false><<<2 * n_pairs, N_THREADS, SMEM2_BYTES, s>>>(tmA, tmB[0], tmB[1], tmB[2], th, ep, num_m,
                                                                              n_tiles_n, gn, d_status);
        return cudaGetLastError() == cudaSuccess ? KVR_OK : KVR_ERR_CUDA;
    }
    const int num_m = (ep.M + BM - 1) / BM;
    const int total = num_m * n_tiles_n;
    const int grid = total < n_sms ? total : n_sms;
    if (ext)
        gemm_tc_kernel<true><<<grid, N_THREADS, SMEM_BYTES, s>>>(tmA, tmB[0], tmB[1], tmB[2], th, ep, num_m, n_tiles_n, gn,
                                                                d_status);
    else
        gemm_tc_kernel<false><<<grid, N_THREADS, SMEM_BYTES, s>>>(tmA, tmB[0], tmB[1], tmB[2], th, ep, num_m, n_tiles_n, gn,
                                                                 d_status);
    return cudaGetLastError() == cudaSuccess ? KVR_OK : KVR_ERR_CUDA;
}

}  // namespace kvr
