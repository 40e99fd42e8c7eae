// Variable-length causal attention prefill over paged K/V on tcgen05.
//
// One CTA = up to 256 consecutive query rows of one request (two sub-tiles A
// and B of 128 rows) x one query head.  Keys/values are visited 128 at a time;
// each 16-slot arena block of a tile arrives by its own TMA box (K and V are
// read through the request's block table, 128-byte swizzle).  Per sub-tile and
// step:  S = Q K^T (SS MMA, fp32 in TMEM)  ->  softmax warps (running max with
// lazy rescale, exp2, bf16 P written back over S in TMEM)  ->  O += P V (TS
// MMA: P from TMEM, V from shared memory, MN-major).  The two sub-tiles
// ping-pong on the tensor pipe (QK_A, QK_B, PV_A, QK_A', PV_B, QK_B', ...) so
// one sub-tile's softmax overlaps the other's MMAs.
//
// Softmax: TWO threads per query row, two 32-key chunks of the step each (chunks
// h and h + 2 for thread h).  A warp issues its instructions in order and a
// special-function instruction holds it for 8 cycles, so a lone warp per
// scheduler cannot overlap the exponentials with the fma/convert work around
// them (measured: 12-13 cycles per element against 8.8-9.2 with two or more
// warps); with two warps of the same sub-tile on every scheduler the phase runs
// close to the special-function unit's rate.  The two threads of a row agree on
// the step's row max through shared memory and a 64-thread named barrier before
// any exponential is taken, so the reference max is exact and a row is never
// redone.  P is handed to the MMA thread in two halves: after the first chunks
// (keys 0..63) the first four K = 16 slices of P V are issued while the softmax
// warps work on keys 64..127.
//
// Warps 0-7: softmax/epilogue of A (warp w: TMEM lanes 32 (w & 3).., key half
// (w >> 2) & 1), 8-15: of B, 16: MMA issue + TMEM alloc, 17: TMA producer (18, 19
// idle: the register hand-over works on whole warpgroups).
// TMEM columns: S_A/P_A 0, O_A 128, S_B/P_B 256, O_B 384.
#include "kvr_internal.h"
#include "kvr_ptx.cuh"

namespace kvr {

namespace {

constexpr int FA_M = 128, FA_N = 128, FA_THREADS = 640;
constexpr int FA_SM_WARPS = 16, FA_MMA_WARP = 16, FA_TMA_WARP = 17;
constexpr int FA_BLOCK = 16;               // arena slots per block (required)
constexpr int BLK_PER_STEP = FA_N / FA_BLOCK;
constexpr int HALF_BYTES = FA_M * 128;     // 128 rows x 64 bf16 (one swizzle-atom column)
constexpr float RESCALE_LOG2 = 8.0f;       // rescale O only when the row max grew by more than 2^8

constexpr int XCHG_BYTES = 2 * 2 * 2 * FA_M * 4;   // [max | sum][sub-tile][key half][row] floats exchanged by a row's two threads
template <int HD> struct FaCfg {
    static constexpr int HALVES = HD / 64;
    static constexpr int TILE_BYTES = HALVES * HALF_BYTES;  // Q sub-tile, K stage or V stage
    static constexpr int SMEM = 6 * TILE_BYTES + 1024 + 256 + XCHG_BYTES;
};

// bf16 x bf16 -> fp32; A K-major (or TMEM), B K-major unless b_mn.
__host__ __device__ constexpr uint32_t fa_idesc(int M, int N, bool b_mn) {
    return (1u << 4) | (1u << 7) | (1u << 10) | (b_mn ? (1u << 16) : 0u) | ((uint32_t)(N >> 3) << 17) |
           ((uint32_t)(M >> 4) << 24);
}
// K and V stages are laid out [8-key group][64-dim half][8 keys][128 bytes]: one TMA box
// brings both halves of a 16-slot block.  K is read K-major (8-key groups `group_bytes`
// apart), V as the MN-major operand: 64-dim atoms 1024 bytes apart (leading offset),
// 8-key groups `group_bytes` apart (stride).
__device__ __forceinline__ uint64_t smem_desc_k_sw128(uint32_t saddr, uint32_t group_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFF) >> 4);
    d |= (uint64_t)1 << 16;
    d |= (uint64_t)(group_bytes >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}
__device__ __forceinline__ uint64_t smem_desc_mn_sw128(uint32_t saddr, uint32_t group_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFF) >> 4);
    d |= (uint64_t)(1024 >> 4) << 16;
    d |= (uint64_t)(group_bytes >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
        "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
          "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
          "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
}
__device__ __forceinline__ float fast_ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack_bf16x2(float a, float b) {
    __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t *>(&h);
}

// A thread's share of a score row: two 32-key chunks of the step (chunks h and h + 2 for key
// half h, so that the first chunks of a row's two threads together cover keys 0..63), both loads
// in flight together; keys after the row's own position are set to -inf on diagonal tiles.
__device__ __forceinline__ void load_score_chunks(uint32_t tS0, uint32_t tS1, uint32_t (&r)[2][32], bool need_mask,
                                                  int key_a, int key_b, int qpos) {
    ptx::tmem_ld32(tS0, r[0]);
    ptx::tmem_ld32(tS1, r[1]);
    ptx::tmem_ld_wait();
    if (need_mask) {
#pragma unroll
        for (int i = 0; i < 32; ++i) {
            if (key_a + i > qpos) r[0][i] = 0xff800000u;   // -inf
            if (key_b + i > qpos) r[1][i] = 0xff800000u;
        }
    }
}
__device__ __forceinline__ float chunks_max(const uint32_t (&r)[2][32]) {
    float m4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
    for (int c = 0; c < 2; ++c)
#pragma unroll
        for (int i = 0; i < 32; ++i) m4[i & 3] = fmaxf(m4[i & 3], __uint_as_float(r[c][i]));
    return fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3]));
}
// Two fp32 lanes per instruction (fma/add on register pairs): halves the issue slots
// the softmax spends beside the exponentials.
__device__ __forceinline__ uint64_t f2_pack(float lo, float hi) {
    uint64_t v;
    asm("mov.b64 %0, {%1, %2};" : "=l"(v) : "f"(lo), "f"(hi));
    return v;
}
__device__ __forceinline__ void f2_unpack(uint64_t v, float &lo, float &hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t f2_fma(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t f2_add(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
// p = 2^(s * scale - msc) for one 32-key chunk: 16 packed bf16 pairs and their fp32 sum.
__device__ __forceinline__ float exp_chunk(const uint32_t (&r)[32], float scale_log2, float msc, uint32_t (&pk)[16]) {
    uint64_t s4[4] = {0ull, 0ull, 0ull, 0ull};
    const uint64_t sc2 = f2_pack(scale_log2, scale_log2), nm2 = f2_pack(-msc, -msc);
#pragma unroll
    for (int i = 0; i < 32; i += 2) {
        float t0, t1;
        f2_unpack(f2_fma(f2_pack(__uint_as_float(r[i]), __uint_as_float(r[i + 1])), sc2, nm2), t0, t1);
        const float p0 = fast_ex2(t0), p1 = fast_ex2(t1);
        s4[(i >> 1) & 3] = f2_add(s4[(i >> 1) & 3], f2_pack(p0, p1));
        pk[i >> 1] = pack_bf16x2(p0, p1);
    }
    float lo, hi;
    f2_unpack(f2_add(f2_add(s4[0], s4[1]), f2_add(s4[2], s4[3])), lo, hi);
    return lo + hi;
}
// 64-thread named barrier shared by the two warps that own the same 32 query rows.
__device__ __forceinline__ void pair_sync(int id) {
    asm volatile("bar.sync %0, 64;" ::"r"(id) : "memory");
}

// One asm block per group of MMAs (a whole Q K^T or P V product of a step): the issuing thread spends a few
// instructions per MMA, which matters because it shares its scheduler with two softmax warps.
__device__ __forceinline__ void mma_group_qk128(uint32_t d_tmem, uint64_t a0, uint64_t b0, uint32_t idesc, uint32_t first_acc) {
    asm volatile(
        "{\n\t.reg .pred pf, pt;\n\t.reg .b64 b;\n\t.reg .b64 a;\n\t"
        "setp.ne.b32 pf, %4, 0;\n\tsetp.eq.b32 pt, 0, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, pf;\n\t"
        "add.u64 a, %1, 2;\n\tadd.u64 b, %2, 2;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], a, b, %3, pt;\n\t"
        "add.u64 a, %1, 4;\n\tadd.u64 b, %2, 4;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], a, b, %3, pt;\n\t"
        "add.u64 a, %1, 6;\n\tadd.u64 b, %2, 6;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], a, b, %3, pt;\n\t"
        "add.u64 a, %1, 1024;\n\tadd.u64 b, %2, 64;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], a, b, %3, pt;\n\t"
        "add.u64 a, %1, 1026;\n\tadd.u64 b, %2, 66;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], a, b, %3, pt;\n\t"
        "add.u64 a, %1, 1028;\n\tadd.u64 b, %2, 68;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], a, b, %3, pt;\n\t"
        "add.u64 a, %1, 1030;\n\tadd.u64 b, %2, 70;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], a, b, %3, pt;\n\t"
        "}"
        ::"r"(d_tmem), "l"(a0), "l"(b0), "r"(idesc), "r"(first_acc)
        : "memory");
}
__device__ __forceinline__ void mma_group_qk64(uint32_t d_tmem, uint64_t a0, uint64_t b0, uint32_t idesc, uint32_t first_acc) {
    asm volatile(
        "{\n\t.reg .pred pf, pt;\n\t.reg .b64 b;\n\t.reg .b64 a;\n\t"
        "setp.ne.b32 pf, %4, 0;\n\tsetp.eq.b32 pt, 0, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, pf;\n\t"
        "add.u64 a, %1, 2;\n\tadd.u64 b, %2, 2;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], a, b, %3, pt;\n\t"
        "add.u64 a, %1, 4;\n\tadd.u64 b, %2, 4;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], a, b, %3, pt;\n\t"
        "add.u64 a, %1, 6;\n\tadd.u64 b, %2, 6;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], a, b, %3, pt;\n\t"
        "}"
        ::"r"(d_tmem), "l"(a0), "l"(b0), "r"(idesc), "r"(first_acc)
        : "memory");
}
// Four K = 16 slices (64 keys) of P V: `a0` = first packed-P column, `b0` = descriptor of the first slice's V rows.
__device__ __forceinline__ void mma_group_pv128_half(uint32_t d_tmem, uint32_t a0, uint64_t b0, uint32_t idesc, uint32_t first_acc) {
    asm volatile(
        "{\n\t.reg .pred pf, pt;\n\t.reg .b64 b;\n\t.reg .b32 a;\n\t"
        "setp.ne.b32 pf, %4, 0;\n\tsetp.eq.b32 pt, 0, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, pf;\n\t"
        "add.u32 a, %1, 8;\n\tadd.u64 b, %2, 256;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [a], b, %3, pt;\n\t"
        "add.u32 a, %1, 16;\n\tadd.u64 b, %2, 512;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [a], b, %3, pt;\n\t"
        "add.u32 a, %1, 24;\n\tadd.u64 b, %2, 768;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [a], b, %3, pt;\n\t"
        "}"
        ::"r"(d_tmem), "r"(a0), "l"(b0), "r"(idesc), "r"(first_acc)
        : "memory");
}
__device__ __forceinline__ void mma_group_pv64_half(uint32_t d_tmem, uint32_t a0, uint64_t b0, uint32_t idesc, uint32_t first_acc) {
    asm volatile(
        "{\n\t.reg .pred pf, pt;\n\t.reg .b64 b;\n\t.reg .b32 a;\n\t"
        "setp.ne.b32 pf, %4, 0;\n\tsetp.eq.b32 pt, 0, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, pf;\n\t"
        "add.u32 a, %1, 8;\n\tadd.u64 b, %2, 128;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [a], b, %3, pt;\n\t"
        "add.u32 a, %1, 16;\n\tadd.u64 b, %2, 256;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [a], b, %3, pt;\n\t"
        "add.u32 a, %1, 24;\n\tadd.u64 b, %2, 384;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [a], b, %3, pt;\n\t"
        "}"
        ::"r"(d_tmem), "r"(a0), "l"(b0), "r"(idesc), "r"(first_acc)
        : "memory");
}
struct FaParams {
    const AttnTile *tiles;
    const int32_t *tables;
    int max_blk, Hq, Hkv, q_dim;
    int k_row0;   // first row of this layer's K plane in the 2-D arena view
    int v_row0;   // ... of its V plane
    __nv_bfloat16 *o;
    int *status;
};

template <int HD>
__global__ void __launch_bounds__(FA_THREADS, 1)
attn_fa_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmKV,
               const FaParams p) {
    using Cfg = FaCfg<HD>;
    constexpr int HALVES = Cfg::HALVES;
    constexpr int TILE = Cfg::TILE_BYTES;
    constexpr int GROUP = HALVES * 1024;   // 8 keys x all halves inside a K/V stage
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sQ[2] = {base, base + TILE};
    const uint32_t sK[2] = {base + 2 * TILE, base + 3 * TILE};
    const uint32_t sV[2] = {base + 4 * TILE, base + 5 * TILE};
    const uint32_t bars = base + 6 * TILE;
    float *xchg = reinterpret_cast<float *>(smem_raw + (bars + 256 - ptx::smem_u32(smem_raw)));   // [2][2][2][FA_M]
    const uint32_t b_qfull = bars, b_kfull = bars + 8, b_vfull = bars + 24, b_kfree = bars + 40,
                   b_vfree = bars + 56, b_vzero = bars + 72, b_sfull = bars + 80, b_pready = bars + 96,
                   b_ofull = bars + 112, b_phi = bars + 128;
    __shared__ uint32_t tmem_base_sh;
    __shared__ int abort_sh;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const AttnTile at = p.tiles[blockIdx.y];
    const int hq = blockIdx.x;
    const int hk = hq / (p.Hq / p.Hkv);
    const int rows_a = min(at.rows, FA_M), rows_b = at.rows - rows_a;
    const bool has_b = rows_b > 0;
    const int kv_len = at.pos0 + at.rows;
    const int n_a = (at.pos0 + rows_a + FA_N - 1) / FA_N;   // steps sub-tile A takes part in
    const int n_b = has_b ? (kv_len + FA_N - 1) / FA_N : 0;
    const int n_steps = has_b ? n_b : n_a;
    const bool tail = (kv_len % FA_N) != 0;

    if (threadIdx.x == 0) {
        abort_sh = 0;
        ptx::mbar_init(b_qfull, 1);
        for (int s = 0; s < 2; ++s) {
            ptx::mbar_init(b_kfull + 8 * s, 1);
            ptx::mbar_init(b_vfull + 8 * s, 1);
            ptx::mbar_init(b_kfree + 8 * s, 1);
            ptx::mbar_init(b_vfree + 8 * s, 1);
            ptx::mbar_init(b_sfull + 8 * s, 1);
            ptx::mbar_init(b_pready + 8 * s, FA_SM_WARPS / 2 * 32);   // P of keys 0..63: one arrival per softmax thread
            ptx::mbar_init(b_phi + 8 * s, FA_SM_WARPS / 2 * 32);      // P of keys 64..127
            ptx::mbar_init(b_ofull + 8 * s, 1);
        }
        ptx::mbar_init(b_vzero, 1);
        ptx::fence_mbar_init();
        ptx::prefetch_tmap(&tmQ);
        ptx::prefetch_tmap(&tmKV);
    }
    if (warp == FA_MMA_WARP) {
        ptx::tmem_alloc(ptx::smem_u32(&tmem_base_sh), 512);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem = tmem_base_sh;
    volatile int *abort_flag = &abort_sh;

    // Registers: the launch gives every thread 96; the warpgroup of the two single-thread roles hands
    // part of its share to the four softmax warpgroups, whose score rows live in registers (the sum
    // stays within the CTA's allocation: 4 x 128 x 104 + 128 x 64 = 640 x 96).  Each role changes its
    // count inside its own branch, so no code is reached with two different counts.
    if (warp >= FA_SM_WARPS) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 64;");
    if (warp == FA_TMA_WARP) {
        // ---------------- TMA producer: the lanes issue a step's boxes together ----------------
        const int32_t *tab = p.tables + (int64_t)at.trow * p.max_blk;
        const int total_blocks = (kv_len + FA_BLOCK - 1) / FA_BLOCK;
        const int my_b = lane;   // block of the step this lane fetches (both 64-dim halves in one box)
        bool ok = !ptx::loads_muted(p.status);   // test hook: no loads at all, every consumer's wait runs out
        if (lane == 0 && ok) {
            ptx::mbar_expect_tx(b_qfull, (has_b ? 2 : 1) * TILE);
            for (int x = 0; x < (has_b ? 2 : 1); ++x)
                for (int h = 0; h < HALVES; ++h)
                    ptx::tma_load_2d(sQ[x] + h * HALF_BYTES, &tmQ, hq * HD + h * 64, at.q_off + x * FA_M, b_qfull);
        }
        for (int j = 0; j < n_steps && ok; ++j) {
            const int s = j & 1;
            const uint32_t ph = (uint32_t)(j >> 1) & 1u;
            const int nblk = min(BLK_PER_STEP, total_blocks - j * BLK_PER_STEP);
            const bool mine = my_b < nblk;
            const int blk = mine ? tab[j * BLK_PER_STEP + my_b] : 0;
            const uint32_t dst_off = my_b * (2 * GROUP);
            if (!ptx::mbar_wait(b_kfree + 8 * s, ph ^ 1u, p.status, abort_flag)) { ok = false; break; }
            if (lane == 0) ptx::mbar_expect_tx(b_kfull + 8 * s, nblk * HALVES * FA_BLOCK * 128);
            __syncwarp();
            if (mine)
                ptx::tma_load_4d((s ? sK[1] : sK[0]) + dst_off, &tmKV, 0, 0, hk * HALVES, (p.k_row0 + blk * FA_BLOCK) >> 3,
                                 b_kfull + 8 * s);
            if (!ptx::mbar_wait(b_vfree + 8 * s, ph ^ 1u, p.status, abort_flag)) { ok = false; break; }
            if (lane == 0) ptx::mbar_expect_tx(b_vfull + 8 * s, nblk * HALVES * FA_BLOCK * 128);
            __syncwarp();
            if (mine)
                ptx::tma_load_4d((s ? sV[1] : sV[0]) + dst_off, &tmKV, 0, 0, hk * HALVES, (p.v_row0 + blk * FA_BLOCK) >> 3,
                                 b_vfull + 8 * s);
            if (tail && j == n_steps - 1) {
                // V rows past the prefix may hold anything (NaN included): zero them so
                // that their zero probabilities cannot poison the PV product.
                if (!ptx::mbar_wait(b_vfull + 8 * s, ph, p.status, abort_flag)) { ok = false; break; }
                const int r0 = kv_len - j * FA_N;
                uint8_t *vst = smem_raw + ((s ? sV[1] : sV[0]) - ptx::smem_u32(smem_raw));
                const int n16 = (FA_N - r0) * HALVES * 8;
                for (int i = lane; i < n16; i += 32) {
                    const int r = r0 + i / (HALVES * 8), h = (i / 8) % HALVES, q = i % 8;
                    *reinterpret_cast<uint4 *>(vst + (r >> 3) * GROUP + h * 1024 + (r & 7) * 128 + q * 16) =
                        make_uint4(0, 0, 0, 0);
                }
                ptx::fence_proxy_async();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(b_vzero);
            }
        }
    } else if (warp == FA_MMA_WARP) {
        // ---------------- MMA issuer ----------------
        // One thread issues every MMA and commit of the CTA; what it does between two MMAs decides how
        // long the tensor pipe idles (a 64-cycle MMA cannot cover a barrier poll), so its loop is kept short.
        if (lane == 0) {
            constexpr uint32_t IDESC_QK = fa_idesc(FA_M, FA_N, false);
            constexpr uint32_t IDESC_PV = fa_idesc(FA_M, HD, true);
            const uint32_t tS[2] = {tmem, tmem + 256}, tO[2] = {tmem + 128, tmem + 384};
            const int n_x[2] = {n_a, n_b};
            bool ok = ptx::mbar_wait(b_qfull, 0, p.status, abort_flag);
            // descriptors are built once; per MMA only the 16-byte address field moves (scalars chosen by a
            // select, not arrays indexed by the stage: an indexed array would live in local memory)
            const uint64_t qd0 = ptx::smem_desc_sw128(sQ[0]), qd1 = ptx::smem_desc_sw128(sQ[1]);
            const uint64_t kd0 = smem_desc_k_sw128(sK[0], GROUP), kd1 = smem_desc_k_sw128(sK[1], GROUP);
            const uint64_t vd0 = smem_desc_mn_sw128(sV[0], GROUP), vd1 = smem_desc_mn_sw128(sV[1], GROUP);
            auto issue_qk = [&](int x, int j) {
                const uint64_t kd = (j & 1) ? kd1 : kd0, qd = x ? qd1 : qd0;
                {
                    if (HD == 128) mma_group_qk128(x ? tmem + 256 : tmem, qd, kd, IDESC_QK, 0);
                    else mma_group_qk64(x ? tmem + 256 : tmem, qd, kd, IDESC_QK, 0);
                    ptx::mma_commit(b_sfull + 8 * x);
                }
            };
            // step 0 scores
            if (ok) ok = ptx::mbar_wait(b_kfull, 0, p.status, abort_flag);
            if (ok) {
                ptx::tc_fence_after();
                issue_qk(0, 0);
                if (has_b) issue_qk(1, 0);
            }
            for (int j = 0; j < n_steps && ok; ++j) {
                const int s = j & 1;
                const uint32_t ph = (uint32_t)(j >> 1) & 1u;
                const uint64_t vd = s ? vd1 : vd0;
                // The loads of this step's V and the next step's K landed long ago: their barriers are
                // polled first, while the previous step's last MMAs still run, so that between the
                // groups below only the wait for P stands.
                // A poll costs its shared-memory round trip even when the phase is long complete, so the three
                // barriers this step starts with are probed back to back (their latencies overlap) and
                // only one that is still pending is waited for.
                const int x_first = j < n_a ? 0 : 1;
                const uint32_t kb_next = b_kfull + 8 * ((j + 1) & 1), kph_next = (uint32_t)((j + 1) >> 1) & 1u;
                const bool v_in = ptx::mbar_try_wait(b_vfull + 8 * s, ph);
                const bool k_in = j + 1 < n_steps ? ptx::mbar_try_wait(kb_next, kph_next) : true;
                const bool p_in = ptx::mbar_try_wait(b_pready + 8 * x_first, (uint32_t)j & 1u);
                if (!v_in && !ptx::mbar_wait(b_vfull + 8 * s, ph, p.status, abort_flag)) { ok = false; break; }
                if (tail && j == n_steps - 1 && !ptx::mbar_wait(b_vzero, 0, p.status, abort_flag)) { ok = false; break; }
                if (!k_in && !ptx::mbar_wait(kb_next, kph_next, p.status, abort_flag)) { ok = false; break; }
#pragma unroll
                for (int x = 0; x < 2; ++x) {
                    if (!ok || j >= n_x[x]) continue;
                    // P_x(j) of keys 0..63 ready (and O_x rescaled) -> O_x += P_x V over those keys, while the
                    // softmax warps still work on keys 64..127; then the same for the second half
                    if (!(x == x_first && p_in) &&
                        !ptx::mbar_wait(b_pready + 8 * x, (uint32_t)j & 1u, p.status, abort_flag)) { ok = false; break; }
                    ptx::tc_fence_after();
                    if (HD == 128) mma_group_pv128_half(tO[x], tS[x], vd, IDESC_PV, j != 0);
                    else mma_group_pv64_half(tO[x], tS[x], vd, IDESC_PV, j != 0);
                    if (!ptx::mbar_wait(b_phi + 8 * x, (uint32_t)j & 1u, p.status, abort_flag)) { ok = false; break; }
                    ptx::tc_fence_after();
                    if (HD == 128) mma_group_pv128_half(tO[x], tS[x] + 32, vd + 1024, IDESC_PV, 1);
                    else mma_group_pv64_half(tO[x], tS[x] + 32, vd + 512, IDESC_PV, 1);
                    if (j == n_x[x] - 1) ptx::mma_commit(b_ofull + 8 * x);
                    // next step's scores for this sub-tile
                    if (j + 1 < n_x[x]) {
                        issue_qk(x, j + 1);
                    }
                }
            }
        }
    }
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 104;");
        // ---------------- softmax + epilogue: two threads per query row ----------------
        const int x = warp >> 3;                    // 0: sub-tile A, 1: sub-tile B
        const int half = (warp >> 2) & 1;           // which 64 keys of a step (and which half of O's columns)
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;        // row inside the sub-tile = TMEM lane
        const int n_mine = x == 0 ? n_a : n_b;
        const int qpos = at.pos0 + x * FA_M + row;  // prefix position of this row
        const bool valid = x * FA_M + row < at.rows;
        const uint32_t lane_sel = (uint32_t)(quarter * 32) << 16;
        const uint32_t tSx = tmem + lane_sel + (x ? 256 : 0), tOx = tmem + lane_sel + (x ? 384 : 128);
        constexpr int OC = HD / 2;                  // my share of O's columns
        const uint32_t tO = tOx + half * OC;
        const int bar_id = 1 + x * 4 + quarter;     // named barrier of this row group's two warps
        float *my_x = xchg + (x * 2 + half) * FA_M + row, *peer_x = xchg + (x * 2 + (half ^ 1)) * FA_M + row;
        const float scale_log2 = rsqrtf((float)HD) * 1.4426950408889634f;
        float m_ref = 0.f, l_sum = 0.f;
        bool ok = true;
        for (int j = 0; j < n_mine; ++j) {
            // After a wait gave up the warp keeps walking its steps, skipping the work but not the pair
            // barrier: its partner warp counts on one barrier call per step.
            if (ok && !ptx::mbar_wait(b_sfull + 8 * x, (uint32_t)j & 1u, p.status, abort_flag)) ok = false;
            if (!ok) { pair_sync(bar_id); continue; }
            ptx::tc_fence_after();
            // The scores of step j are complete, so (in-order tensor pipe) every earlier MMA is too:
            // both sub-tiles are done reading K(j) and V(j - 1).  One thread of the sub-tile that takes
            // part in every step hands the two stages back to the producer, which spares the
            // MMA-issuing thread two commits per step.
            if (x == (has_b ? 1 : 0) && (warp & 7) == 0 && lane == 0) {
                ptx::mbar_arrive(b_kfree + 8 * (j & 1));
                if (j > 0) ptx::mbar_arrive(b_vfree + 8 * ((j - 1) & 1));
            }
            const int key_a = j * FA_N + 32 * half, key_b = key_a + 64;   // my two 32-key chunks
            // this warp's smallest position is that of lane 0
            const bool need_mask = key_b + 31 > at.pos0 + x * FA_M + quarter * 32;
            uint32_t r[2][32], pk[16];
            load_score_chunks(tSx + 32 * half, tSx + 32 * half + 64, r, need_mask, key_a, key_b, qpos);
            // Row max of the step: mine, then the partner's through shared memory.  All four loads of the
            // row are complete on both sides of the barrier, so either thread may now overwrite score
            // columns the other one read (P's columns lie over the scores of keys 0..63).
            *my_x = chunks_max(r);
            pair_sync(bar_id);
            const float mx = fmaxf(*my_x, *peer_x);
            // Reference max: moved only when the row max outgrew it by more than 2^8 (key 0 is visible to
            // every row, so step 0's is finite).  Both threads of a row take the same decision.
            const bool grow = j == 0 || (mx - m_ref) * scale_log2 > RESCALE_LOG2;
            if (__any_sync(0xffffffffu, grow && j > 0)) {
                const float corr = grow ? fast_ex2((m_ref - mx) * scale_log2) : 1.f;
                l_sum *= corr;
#pragma unroll 1
                for (int c = 0; c < OC; c += 16) {   // rare: small chunks keep the registers for the score row
                    uint32_t o[16];
                    ptx::tmem_ld16(tO + c, o);
                    ptx::tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 16; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * corr);
                    tmem_st16(tO + c, o);
                }
            }
            if (grow) m_ref = mx;
            const float msc = m_ref * scale_log2;
            // First chunks (keys 0..63 between the two threads): bf16 P over the scores, 16 packed columns
            // per chunk, handed to the MMA thread before the second chunks are touched.
            l_sum += exp_chunk(r[0], scale_log2, msc, pk);
            tmem_st16(tSx + 16 * half, pk);
            ptx::tmem_st_wait();
            ptx::tc_fence_before();
            ptx::mbar_arrive(b_pready + 8 * x);
            l_sum += exp_chunk(r[1], scale_log2, msc, pk);
            tmem_st16(tSx + 16 * half + 32, pk);
            ptx::tmem_st_wait();
            ptx::tc_fence_before();
            ptx::mbar_arrive(b_phi + 8 * x);
        }
        // row sum = both halves' (slots of their own: the partner may still be reading the last max)
        my_x[4 * FA_M] = l_sum;
        pair_sync(bar_id);
        l_sum += peer_x[4 * FA_M];
        if (ok && n_mine > 0 && ptx::mbar_wait(b_ofull + 8 * x, 0, p.status, abort_flag)) {
            ptx::tc_fence_after();
            const float inv = 1.0f / l_sum;
            __nv_bfloat16 *dst = p.o + (int64_t)(at.q_off + x * FA_M + row) * p.q_dim + hq * HD + half * OC;
#pragma unroll 1
            for (int c = 0; c < OC; c += 32) {
                uint32_t r[32];
                ptx::tmem_ld32(tO + c, r);
                ptx::tmem_ld_wait();
                if (!valid) continue;
#pragma unroll
                for (int i = 0; i < 32; i += 8)
                    *reinterpret_cast<uint4 *>(dst + c + i) = make_uint4(
                        pack_bf16x2(__uint_as_float(r[i]) * inv, __uint_as_float(r[i + 1]) * inv),
                        pack_bf16x2(__uint_as_float(r[i + 2]) * inv, __uint_as_float(r[i + 3]) * inv),
                        pack_bf16x2(__uint_as_float(r[i + 4]) * inv, __uint_as_float(r[i + 5]) * inv),
                        pack_bf16x2(__uint_as_float(r[i + 6]) * inv, __uint_as_float(r[i + 7]) * inv));
            }
        }
    }
    ptx::tc_fence_before();
    __syncthreads();
    if (warp == FA_MMA_WARP) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem, 512);
    }
}

}  // namespace

int attn_fa_init(int device) {
    (void)device;
    if (cudaFuncSetAttribute(attn_fa_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, FaCfg<128>::SMEM) !=
            cudaSuccess ||
        cudaFuncSetAttribute(attn_fa_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, FaCfg<64>::SMEM) !=
            cudaSuccess)
        return KVR_ERR_CUDA;
    return KVR_OK;
}

int launch_attn_fa(const CUtensorMap &tmQ, const CUtensorMap &tmKV, const AttnTile *tiles, int n_tiles,
                   const int32_t *tables, int max_blk, const ModelDims &md, const ArenaView &av, int layer,
                   __nv_bfloat16 *o, int *d_status, cudaStream_t s) {
    if (n_tiles <= 0) return KVR_OK;
    if (n_tiles > 65535 || av.block_size != FA_BLOCK) return KVR_ERR_UNSUPPORTED;
    const int64_t slots = (int64_t)av.num_blocks * av.block_size;
    const int64_t k_row0 = (int64_t)layer * 2 * slots;
    if (k_row0 + 2 * slots >= ((int64_t)1 << 31)) return KVR_ERR_UNSUPPORTED;
    FaParams p;
    p.tiles = tiles; p.tables = tables; p.max_blk = max_blk; p.Hq = md.Hq; p.Hkv = md.Hkv; p.q_dim = md.q_dim;
    p.k_row0 = (int)k_row0; p.v_row0 = (int)(k_row0 + slots); p.o = o; p.status = d_status;
    dim3 grid(md.Hq, n_tiles);
    if (md.hd == 128)
        attn_fa_kernel<128><<<grid, FA_THREADS, FaCfg<128>::SMEM, s>>>(tmQ, tmKV, p);
    else if (md.hd == 64)
        attn_fa_kernel<64><<<grid, FA_THREADS, FaCfg<64>::SMEM, s>>>(tmQ, tmKV, p);
    else
        return KVR_ERR_UNSUPPORTED;
    return cudaGetLastError() == cudaSuccess ? KVR_OK : KVR_ERR_CUDA;
}

}  // namespace kvr
