// Device steps of the handover that precede the rebuild: the lightweight GPU
// health check and the flush of the KV-cache pool (paper Sec. 4.2, step 2).
#include "kvr_internal.h"

#include <chrono>
#include <thread>

namespace kvr {

namespace {

// ---- flush: every byte of the arena <- a 32-bit word, 16-byte stores, HBM-bound ----
template <int UNROLL>
__global__ void __launch_bounds__(256) arena_flush_kernel(uint4 *__restrict__ dst, int64_t n16, uint32_t word) {
    const uint4 v = make_uint4(word, word, word, word);
    // each block walks contiguous spans of UNROLL x 256 x 16 bytes
    const int64_t span = (int64_t)UNROLL * blockDim.x;
    for (int64_t base = (int64_t)blockIdx.x * span; base < n16; base += (int64_t)gridDim.x * span) {
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            const int64_t i = base + (int64_t)u * blockDim.x + threadIdx.x;
            if (i < n16) __stcs(dst + i, v);
        }
    }
}

// ---- probe: ALU + shared memory + global memory + cross-SM visibility, bounded wait ----
__device__ __forceinline__ uint32_t xorshift32(uint32_t x) {
    x ^= x << 13;
    x ^= x >> 17;
    x ^= x << 5;
    return x;
}

// `epoch` is a word no earlier probe of this flag array has published (the context counts its
// calls), so a flag left behind by a previous call can never satisfy this call's wait.
__global__ void __launch_bounds__(PROBE_THREADS) probe_kernel(uint32_t seed, uint32_t epoch, uint32_t *flags,
                                                              uint32_t *out, int *status, long long limit_cycles,
                                                              int publish) {
    __shared__ uint32_t red[PROBE_THREADS];
    const uint32_t b = blockIdx.x, t = threadIdx.x;
    uint32_t x = seed ^ (b * 0x9E3779B9u) ^ (t * 0x85EBCA6Bu);
    if (x == 0) x = 1;
    for (int i = 0; i < PROBE_ITERS; ++i) x = xorshift32(x) + 0x9E3779B9u;   // not linear over GF(2)
    red[t] = x;
    __syncthreads();
    for (int s = PROBE_THREADS / 2; s > 0; s >>= 1) {
        if (t < s) red[t] += red[t + s];
        __syncthreads();
    }
    if (t == 0) {
        out[b] = red[0];
        __threadfence();
        if (publish) atomicExch(&flags[b], epoch);
        // the neighbour block must become visible within the limit; a wait that runs out
        // is reported through the status word, never by spinning on
        const uint32_t nb = (b + 1) % gridDim.x;
        const long long t0 = clock64();
        while (atomicAdd(&flags[nb], 0u) != epoch) {
            if (clock64() - t0 > limit_cycles) {
                atomicExch(status, KVR_ERR_DEVICE_TIMEOUT);
                break;
            }
            __nanosleep(200);
        }
    }
}

}  // namespace

int launch_arena_flush(void *arena, size_t bytes, uint32_t word, int n_sms, cudaStream_t s) {
    if (bytes % 16) return KVR_ERR_UNSUPPORTED;
    const int64_t n16 = (int64_t)(bytes / 16);
    if (n16 == 0) return KVR_OK;
    // 16 blocks per SM, 8 x 4 KB contiguous per block visit, streaming stores: measured 6.9 TB/s
    arena_flush_kernel<8><<<n_sms * 16, 256, 0, s>>>((uint4 *)arena, n16, word);
    return cudaGetLastError() == cudaSuccess ? KVR_OK : KVR_ERR_CUDA;
}

int launch_probe(uint32_t seed, uint32_t epoch, uint32_t *flags, uint32_t *out, int *status, int blocks,
                 long long limit_cycles, int publish, cudaStream_t s) {
    probe_kernel<<<blocks, PROBE_THREADS, 0, s>>>(seed, epoch, flags, out, status, limit_cycles, publish);
    return cudaGetLastError() == cudaSuccess ? KVR_OK : KVR_ERR_CUDA;
}

}  // namespace kvr
