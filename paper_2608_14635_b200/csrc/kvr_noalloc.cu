// kv_readback_noalloc: the read-back gather for callers that must not allocate.
//
// Its staging lives in a fixed array inside the library's device image instead
// of a caller-bound workspace, so the call needs no context, no workspace and
// no allocation of any kind.  The array exists once per GPU that loads the
// library, for the life of the process, and is shared by every call.
#include "kvr_internal.h"

#include <mutex>

namespace {

constexpr size_t TABLE_BYTES = (size_t)KVR_NOALLOC_MAX_BLOCKS * sizeof(int32_t);      // 16 KiB
constexpr size_t PLANE_BYTES = (size_t)KVR_NOALLOC_MAX_PLANE_BYTES;                    // 2 MiB each for K and V
constexpr size_t SCRATCH_BYTES = TABLE_BYTES + 2 * PLANE_BYTES;
constexpr int MAX_DEVICES = 64;

// Device-resident staging: [block table | dense K rows | dense V rows].
static __device__ __align__(256) unsigned char g_noalloc_scratch[SCRATCH_BYTES];

// In host code `g_noalloc_scratch` is only a handle for the runtime, not an
// address a kernel may use: the device address is looked up once per device.
std::mutex g_mu;
unsigned char *g_dev_ptr[MAX_DEVICES] = {};

__global__ void readback_noalloc_kernel(const uint4 *__restrict__ arena_k, int64_t kv_stride_v, int row_v,
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

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; prev = -1; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    }
    ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

}  // namespace

extern "C" int kv_readback_noalloc(const void *arena_dev, const kv_arena_geometry *g, int32_t layer,
                                   const int32_t *table, int32_t n, void *k_out, void *v_out, void *stream_v) {
    if (!arena_dev || !g || n < 0) return KVR_ERR_INVALID_ARG;
    if (g->block_size <= 0 || g->num_blocks <= 0 || g->n_layers <= 0 || g->n_kv_heads <= 0 || g->head_dim <= 0 ||
        (g->dtype != KVR_BF16 && g->dtype != KVR_FP32))
        return KVR_ERR_INVALID_ARG;
    if (layer < 0 || layer >= g->n_layers) return KVR_ERR_INVALID_ARG;
    if (n == 0) return KVR_OK;
    if (!table || !k_out || !v_out) return KVR_ERR_INVALID_ARG;
    const size_t es = g->dtype == KVR_FP32 ? 4 : 2;
    const size_t row_bytes = (size_t)g->n_kv_heads * g->head_dim * es;
    if (row_bytes % 16 || ((uintptr_t)arena_dev) % 16) return KVR_ERR_UNSUPPORTED;
    const int need = (n + g->block_size - 1) / g->block_size;
    // the fixed staging bounds what one call can read back
    if (need > KVR_NOALLOC_MAX_BLOCKS || (size_t)n * row_bytes > PLANE_BYTES) return KVR_ERR_WORKSPACE;
    for (int j = 0; j < need; ++j) {
        if (table[j] == -1) return KVR_ERR_TABLE_TOO_SHORT;
        if (table[j] < 0 || table[j] >= g->num_blocks) return KVR_ERR_BLOCK_OOB;
    }
    cudaPointerAttributes attr;
    if (cudaPointerGetAttributes(&attr, arena_dev) != cudaSuccess || attr.type != cudaMemoryTypeDevice)
        return KVR_ERR_INVALID_ARG;
    const int dev = attr.device;
    if (dev < 0 || dev >= MAX_DEVICES) return KVR_ERR_UNSUPPORTED;
    DeviceGuard guard(dev);
    if (!guard.ok) return KVR_ERR_CUDA;
    {
        // There is no arena_bytes argument, so the extent of the allocation that holds arena_dev is
        // asked of the driver (a query, not an allocation): the layer's K and V planes must lie
        // inside it, otherwise a wrong geometry would turn into an out-of-range device read.
        typedef CUresult (*RangeFn)(CUdeviceptr *, size_t *, CUdeviceptr);
        static RangeFn range_fn = nullptr;
        {
            std::lock_guard<std::mutex> lock(g_mu);
            if (!range_fn) {
                void *fn = nullptr;
                cudaDriverEntryPointQueryResult qres;
                if (cudaGetDriverEntryPoint("cuMemGetAddressRange", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
                    qres != cudaDriverEntryPointSuccess || !fn)
                    return KVR_ERR_CUDA;
                range_fn = (RangeFn)fn;
            }
        }
        CUdeviceptr abase = 0;
        size_t asize = 0;
        if (range_fn(&abase, &asize, (CUdeviceptr)(uintptr_t)arena_dev) != CUDA_SUCCESS) return KVR_ERR_INVALID_ARG;
        const size_t plane_bytes = (size_t)g->num_blocks * g->block_size * row_bytes;
        const size_t end = (size_t)((uintptr_t)arena_dev - (uintptr_t)abase) + ((size_t)layer + 1) * 2 * plane_bytes;
        if (end > asize) return KVR_ERR_INVALID_ARG;
    }

    unsigned char *scratch = nullptr;
    {
        // first call on this device: resolve the array's device address (with
        // that device current); later calls reuse it
        std::lock_guard<std::mutex> lock(g_mu);
        if (!g_dev_ptr[dev]) {
            void *ptr = nullptr;
            if (cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess || !ptr) return KVR_ERR_CUDA;
            g_dev_ptr[dev] = (unsigned char *)ptr;
        }
        scratch = g_dev_ptr[dev];
    }
    cudaStream_t s = (cudaStream_t)stream_v;
    int32_t *d_table = (int32_t *)scratch;
    unsigned char *d_k = scratch + TABLE_BYTES, *d_v = d_k + PLANE_BYTES;
    const size_t dense = (size_t)n * row_bytes;
    if (cudaMemcpyAsync(d_table, table, (size_t)need * sizeof(int32_t), cudaMemcpyHostToDevice, s) != cudaSuccess)
        return KVR_ERR_CUDA;
    const int64_t slots = (int64_t)g->num_blocks * g->block_size;
    const int row_v = (int)(row_bytes / 16);
    const int64_t kv_stride_v = slots * row_v;
    const uint4 *plane = (const uint4 *)arena_dev + (int64_t)layer * 2 * kv_stride_v;
    const int64_t total = (int64_t)n * row_v;
    readback_noalloc_kernel<<<(unsigned)((total + 255) / 256), 256, 0, s>>>(plane, kv_stride_v, row_v, d_table,
                                                                            g->block_size, n, (uint4 *)d_k,
                                                                            (uint4 *)d_v);
    // From here on work may be in flight on the shared array: every return waits for the stream,
    // so that a failed call cannot race with the next one.
    bool ok = cudaGetLastError() == cudaSuccess;
    ok = ok && cudaMemcpyAsync(k_out, d_k, dense, cudaMemcpyDeviceToHost, s) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(v_out, d_v, dense, cudaMemcpyDeviceToHost, s) == cudaSuccess;
    const bool synced = cudaStreamSynchronize(s) == cudaSuccess;
    return ok && synced ? KVR_OK : KVR_ERR_CUDA;
}
