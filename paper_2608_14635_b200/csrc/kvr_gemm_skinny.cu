// Weight-streaming GEMM for a handful of activation rows (the R final-token rows of
// kv_resume_logits, R <= 128):  out[r, n] = sum_k X[r, k] W[n, k].
// With so few rows the product is bound by reading W once from HBM, so the grid is cut
// along the weight rows (and, for matrices with few rows, along K) instead of along R:
//   - the operands are swapped on the tensor core: the 128 weight rows of a CTA's tile are
//     the MMA's M, the requests are its N (padded to a multiple of 16), so the accumulator
//     in TMEM is out^T: lane = weight row n, column = request r, and a warp's store of one
//     column writes 32 consecutive n of one output row;
//   - a work item is (128-row tile, split); a split covers a contiguous range of 64-wide K
//     blocks and writes its fp32 partial product to out + split * split_stride, which the
//     consumer kernel sums in a fixed order (no atomics, run-to-run identical);
//   - persistent CTAs, one per SM, take items round-robin; a TMA ring of nine 24 KB stages
//     (five 40 KB stages for the SwiGLU pair; six and four when there are more than 64
//     rows) keeps about 150 KB of weight bytes in flight per SM across items - the kernel
//     is bound by how many bytes it keeps in flight, not by DRAM or L2 throughput - and two accumulator buffers in TMEM let the epilogue of one item
//     run under the loads and MMAs of the next.
// Warp 0 = TMA producer, warp 1 = MMA issuer and TMEM owner, warps 2..5 = epilogue.
// Every wait is bounded through the context's status block, as in the large GEMM.
#include "kvr_internal.h"
#include "kvr_ptx.cuh"

namespace kvr {

namespace {

constexpr int SK_ROWS = 128, SK_BK = 64, SK_UMMA_K = 16;
constexpr int SK_TILE_BYTES = SK_ROWS * SK_BK * 2;   // one 128 x 64 bf16 box
constexpr int SK_THREADS = 192;

// XROWS: rows of the activation box (64 when the call has at most 64 rows: the smaller box leaves
// shared memory for more stages, i.e. more weight bytes in flight)
template <bool SWIGLU, int XROWS>
struct SkCfg {
    static constexpr int N_W = SWIGLU ? 2 : 1;                       // weight boxes per stage
    static constexpr int X_BYTES = XROWS * SK_BK * 2;
    static constexpr int STAGE_BYTES = N_W * SK_TILE_BYTES + X_BYTES;   // weights, then the activation box
    static constexpr int STAGES = (220 * 1024) / STAGE_BYTES;        // 128 rows: 6 / 4 (pair), 64 rows: 9 / 5
    static constexpr int ACC_COLS = SWIGLU ? 256 : 128;              // one accumulator buffer (gate | up)
    static constexpr int TMEM_COLS = 2 * ACC_COLS;                   // two buffers: epilogue overlaps the next item
    static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 /*align slack*/ + 256 /*barriers*/;
};

// Work item w of a launch: tile = w % n_tiles, split = w / n_tiles (neighbouring CTAs share a K range of X).
struct SkItem { int tile, kb0, kb1; int split; };
__device__ __forceinline__ SkItem sk_item(int w, int n_tiles, int n_split, int num_k) {
    SkItem it;
    it.split = w / n_tiles;
    it.tile = w - it.split * n_tiles;
    it.kb0 = (int)((int64_t)it.split * num_k / n_split);
    it.kb1 = (int)((int64_t)(it.split + 1) * num_k / n_split);
    return it;
}

template <bool SWIGLU, int XROWS>
__global__ void __launch_bounds__(SK_THREADS, 1)
gemm_skinny_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmW0,
                   const __grid_constant__ CUtensorMap tmW1, const SkinnyArgs a, int n_split, int *status) {
    using Cfg = SkCfg<SWIGLU, XROWS>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = ptx::smem_u32(smem_raw);
    const uint32_t tiles = (raw + 1023u) & ~1023u;
    const uint32_t bars = tiles + Cfg::STAGES * Cfg::STAGE_BYTES;
    // barrier addresses: full[s], empty[s], tmem_full[2], tmem_empty[2]
    const uint32_t full0 = bars, empty0 = bars + 8 * Cfg::STAGES, tfull0 = bars + 16 * Cfg::STAGES,
                   tempty0 = bars + 16 * Cfg::STAGES + 16;
    __shared__ uint32_t tmem_base_sh;
    __shared__ int abort_sh;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        abort_sh = 0;
        for (int s = 0; s < Cfg::STAGES; ++s) {
            ptx::mbar_init(full0 + 8 * s, 1);
            ptx::mbar_init(empty0 + 8 * s, 1);
        }
        for (int b = 0; b < 2; ++b) {
            ptx::mbar_init(tfull0 + 8 * b, 1);
            ptx::mbar_init(tempty0 + 8 * b, 4);
        }
        ptx::fence_mbar_init();
        ptx::prefetch_tmap(&tmX);
        ptx::prefetch_tmap(&tmW0);
    }
    if (warp == 1) {
        ptx::tmem_alloc(ptx::smem_u32(&tmem_base_sh), Cfg::TMEM_COLS);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = tmem_base_sh;
    volatile int *abort_flag = &abort_sh;
    // everything above is local to the CTA and may run while the kernel before this one drains
    grid_dependency_wait();
    grid_launch_dependents();

    const int n_tiles = (a.N + SK_ROWS - 1) / SK_ROWS;
    const int total = n_tiles * n_split;
    const int num_k = (a.K + SK_BK - 1) / SK_BK;
    const int n_pad = a.R <= 16 ? 16 : ((a.R + 15) & ~15);
    // a split with no K block (more splits than blocks) has a zero partial product: the producer and the MMA
    // thread skip the item, the epilogue stores zeros without touching an accumulator

    if (warp == 0) {
        if (lane == 0 && !ptx::loads_muted(status)) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int w = blockIdx.x; w < total && ok; w += gridDim.x) {
                const SkItem it = sk_item(w, n_tiles, n_split, num_k);
                for (int kb = it.kb0; kb < it.kb1; ++kb) {
                    if (!ptx::mbar_wait(empty0 + 8 * stage, phase ^ 1u, status, abort_flag)) { ok = false; break; }
                    const uint32_t fb = full0 + 8 * stage;
                    const uint32_t sa = tiles + stage * Cfg::STAGE_BYTES;
                    ptx::mbar_expect_tx(fb, Cfg::STAGE_BYTES);
                    ptx::tma_load_2d(sa, &tmW0, kb * SK_BK, it.tile * SK_ROWS, fb);
                    if (SWIGLU) ptx::tma_load_2d(sa + SK_TILE_BYTES, &tmW1, kb * SK_BK, it.tile * SK_ROWS, fb);
                    ptx::tma_load_2d(sa + Cfg::N_W * SK_TILE_BYTES, &tmX, kb * SK_BK, 0, fb);
                    if (++stage == Cfg::STAGES) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = ptx::idesc_bf16(SK_ROWS, n_pad);
            int stage = 0, acc = 0;
            uint32_t phase = 0, acc_phase = 0;
            bool ok = true;
            for (int w = blockIdx.x; w < total && ok; w += gridDim.x) {
                const SkItem it = sk_item(w, n_tiles, n_split, num_k);
                if (it.kb1 <= it.kb0) continue;
                if (!ptx::mbar_wait(tempty0 + 8 * acc, acc_phase ^ 1u, status, abort_flag)) break;
                ptx::tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * Cfg::ACC_COLS;
                for (int kb = it.kb0; kb < it.kb1; ++kb) {
                    if (!ptx::mbar_wait(full0 + 8 * stage, phase, status, abort_flag)) { ok = false; break; }
                    ptx::tc_fence_after();
                    const uint32_t sa = tiles + stage * Cfg::STAGE_BYTES;
                    const uint64_t dw0 = ptx::smem_desc_sw128(sa);
                    const uint64_t dw1 = ptx::smem_desc_sw128(sa + SK_TILE_BYTES);
                    const uint64_t dx = ptx::smem_desc_sw128(sa + Cfg::N_W * SK_TILE_BYTES);
#pragma unroll
                    for (int kk = 0; kk < SK_BK / SK_UMMA_K; ++kk) {
                        const uint32_t accum = (kb > it.kb0 || kk > 0) ? 1u : 0u;
                        ptx::mma_bf16_ss(d_tmem, dw0 + 2 * kk, dx + 2 * kk, idesc, accum);
                        if (SWIGLU) ptx::mma_bf16_ss(d_tmem + 128, dw1 + 2 * kk, dx + 2 * kk, idesc, accum);
                    }
                    ptx::mma_commit(empty0 + 8 * stage);
                    if (++stage == Cfg::STAGES) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                ptx::mma_commit(tfull0 + 8 * acc);
                if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
            }
        }
    } else {
        const int quarter = warp & 3;   // the 32 TMEM lanes this warp may read
        int acc = 0;
        uint32_t acc_phase = 0;
        for (int w = blockIdx.x; w < total; w += gridDim.x) {
            const SkItem it = sk_item(w, n_tiles, n_split, num_k);
            const bool empty = it.kb1 <= it.kb0;
            const int n = it.tile * SK_ROWS + quarter * 32 + lane;
            if (!empty) {
                if (!ptx::mbar_wait(tfull0 + 8 * acc, acc_phase, status, abort_flag)) break;
                ptx::tc_fence_after();
            }
            const uint32_t tacc = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * Cfg::ACC_COLS;
#pragma unroll 1
            for (int c = 0; c < n_pad; c += 16) {
                uint32_t g[16], u[16];
                if (!empty) {
                    ptx::tmem_ld16(tacc + c, g);
                    if (SWIGLU) ptx::tmem_ld16(tacc + 128 + c, u);
                    ptx::tmem_ld_wait();
                } else {
#pragma unroll
                    for (int j = 0; j < 16; ++j) g[j] = u[j] = 0u;
                }
                if (n >= a.N) {
                    // rows of the last tile past the matrix: nothing to store
                } else if (SWIGLU) {
                    __nv_bfloat16 *dst = a.out_bf16 + n;
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        if (c + j < a.R) {
                            const float gv = __uint_as_float(g[j]);
                            const float sv = gv / (1.0f + __expf(-gv));
                            dst[(int64_t)(c + j) * a.ld_bf16] = __float2bfloat16_rn(sv * __uint_as_float(u[j]));
                        }
                    }
                } else {
                    float *dst = a.out_f32 + (int64_t)it.split * a.split_stride + n;
#pragma unroll
                    for (int j = 0; j < 16; ++j)
                        if (c + j < a.R) dst[(int64_t)(c + j) * a.ldo] = __uint_as_float(g[j]);
                }
                __syncwarp();
            }
            if (!empty) {
                ptx::tc_fence_before();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(tempty0 + 8 * acc);
                if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
            }
        }
    }
    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem_base, Cfg::TMEM_COLS);
    }
}

}  // namespace

template <bool SWIGLU, int XROWS>
static bool sk_set_smem() {
    return cudaFuncSetAttribute(gemm_skinny_kernel<SWIGLU, XROWS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                SkCfg<SWIGLU, XROWS>::SMEM_BYTES) == cudaSuccess;
}

int gemm_skinny_init(int device) {
    (void)device;
    static_assert(SkCfg<false, 64>::SMEM_BYTES <= 227 * 1024 && SkCfg<true, 64>::SMEM_BYTES <= 227 * 1024 &&
                  SkCfg<false, 128>::SMEM_BYTES <= 227 * 1024 && SkCfg<true, 128>::SMEM_BYTES <= 227 * 1024, "smem");
    return sk_set_smem<false, 64>() && sk_set_smem<true, 64>() && sk_set_smem<false, 128>() && sk_set_smem<true, 128>()
               ? KVR_OK
               : KVR_ERR_CUDA;
}

// One wave of CTAs where the matrix has fewer 128-row tiles than the GPU has SMs.
int gemm_skinny_splits(int N, int K, int n_sms) {
    const int tiles = (N + SK_ROWS - 1) / SK_ROWS, num_k = (K + SK_BK - 1) / SK_BK;
    int s = n_sms / (tiles > 0 ? tiles : 1);
    if (s > GEMM_SKINNY_MAX_SPLITS) s = GEMM_SKINNY_MAX_SPLITS;
    if (s > num_k) s = num_k;
    return s < 1 ? 1 : s;
}

int launch_gemm_skinny(const CUtensorMap &tmX, const CUtensorMap &tmW0, const CUtensorMap *tmW1,
                       const SkinnyArgs &a, int x_rows, int splits, int *d_status, int n_sms, cudaStream_t s,
                       bool pdl) {
    if (a.R <= 0 || a.N <= 0) return KVR_OK;
    if (a.R > GEMM_SKINNY_MAX_ROWS || a.K <= 0 || splits < 1 || splits > GEMM_SKINNY_MAX_SPLITS)
        return KVR_ERR_UNSUPPORTED;
    const int n_split = tmW1 ? 1 : splits;   // the SwiGLU pair needs whole sums before its nonlinearity
    const int total = (a.N + SK_ROWS - 1) / SK_ROWS * n_split;
    const int grid = total < n_sms ? total : n_sms;
    // x_rows = rows of tmX's box: 64 (R <= 64) or 128
    if (x_rows == 64 && a.R <= 64) {
        if (tmW1)
            launch_kernel(gemm_skinny_kernel<true, 64>, dim3(grid), dim3(SK_THREADS), SkCfg<true, 64>::SMEM_BYTES, s, pdl,
                          tmX, tmW0, *tmW1, a, n_split, d_status);
        else
            launch_kernel(gemm_skinny_kernel<false, 64>, dim3(grid), dim3(SK_THREADS), SkCfg<false, 64>::SMEM_BYTES, s,
                          pdl, tmX, tmW0, tmW0, a, n_split, d_status);
    } else if (x_rows == 128) {
        if (tmW1)
            launch_kernel(gemm_skinny_kernel<true, 128>, dim3(grid), dim3(SK_THREADS), SkCfg<true, 128>::SMEM_BYTES, s,
                          pdl, tmX, tmW0, *tmW1, a, n_split, d_status);
        else
            launch_kernel(gemm_skinny_kernel<false, 128>, dim3(grid), dim3(SK_THREADS), SkCfg<false, 128>::SMEM_BYTES, s,
                          pdl, tmX, tmW0, tmW0, a, n_split, d_status);
    } else {
        return KVR_ERR_UNSUPPORTED;
    }
    return cudaGetLastError() == cudaSuccess ? KVR_OK : KVR_ERR_CUDA;
}

}  // namespace kvr
