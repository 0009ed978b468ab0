// Device status word, status strings and the popcount-pipe micro-benchmark.
#include <atomic>

#include "common.cuh"

namespace bs {

__device__ int g_status = 0;

int* status_device_ptr()
{
    int* p = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_status) != cudaSuccess) return nullptr;
    return p;
}

// Multiprocessor count of the current device.  Tile plans depend on it, so it is kept per device ordinal: a process
// that drives GPUs of different sizes gets the right plan on each.
int device_sm_count()
{
    constexpr int kMax = 64;
    static std::atomic<int> cache[kMax];
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0) { cudaGetLastError(); return 0; }
    if (dev < kMax) {
        const int c = cache[dev].load(std::memory_order_relaxed);
        if (c > 0) return c;
    }
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) { cudaGetLastError(); return 0; }
    if (dev < kMax) cache[dev].store(sms, std::memory_order_relaxed);
    return sms;
}

// Register-only chains of acc += popc(x & y).  Operands change every round so nothing folds.
__global__ void __launch_bounds__(256) popc_rate_kernel(int iters, unsigned seed, int* sink)
{
    unsigned x[8], acc[8];
    unsigned y = seed ^ (threadIdx.x * 2654435761u + blockIdx.x);
#pragma unroll
    for (int k = 0; k < 8; ++k) { x[k] = y * (2 * k + 3) + k; acc[k] = 0; }
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int u = 0; u < 4; ++u) {
#pragma unroll
            for (int k = 0; k < 8; ++k) acc[k] += __popc(x[k] & y);
            y = y * 1664525u + 1013904223u;
        }
    }
    unsigned total = 0;
#pragma unroll
    for (int k = 0; k < 8; ++k) total += acc[k];
    if (total == 0xFFFFFFFFu) atomicOr(sink, 0);   // never true in practice; keeps the chains alive
}

// L2 prefetch of up to 64 buffers: one thread per 4 KB piece issues a bulk prefetch, which returns at once; the copy
// into L2 proceeds while the following kernels of the stream run.
struct PrefetchList {
    const unsigned char* ptr[64];
    unsigned long long bytes[64];      // multiples of 16
};

__global__ void l2_prefetch_kernel(const __grid_constant__ PrefetchList list)
{
    const unsigned char* base = list.ptr[blockIdx.y];
    const unsigned long long total = list.bytes[blockIdx.y];
    const unsigned long long piece = 4096;
    for (unsigned long long off = (static_cast<unsigned long long>(blockIdx.x) * blockDim.x + threadIdx.x) * piece; off < total;
         off += static_cast<unsigned long long>(gridDim.x) * blockDim.x * piece) {
        const unsigned long long left = total - off;
        const unsigned n = static_cast<unsigned>(left < piece ? left : piece);
        asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(base + off), "r"(n) : "memory");
    }
}

}  // namespace bs

extern "C" int bs_l2_prefetch(const void* const* buffers, const size_t* bytes, int count, void* stream)
{
    if (count < 0 || (count > 0 && (!buffers || !bytes))) return BS_ERR_INVALID_ARG;
    for (int i = 0; i < count; ++i)
        if (!buffers[i] || !bs::aligned16(buffers[i])) return buffers[i] ? BS_ERR_ALIGNMENT : BS_ERR_INVALID_ARG;
    for (int first = 0; first < count; first += 64) {
        bs::PrefetchList list{};
        const int n = count - first < 64 ? count - first : 64;
        size_t largest = 0;
        for (int i = 0; i < n; ++i) {
            list.ptr[i] = static_cast<const unsigned char*>(buffers[first + i]);
            list.bytes[i] = bytes[first + i] & ~static_cast<size_t>(15);
            if (bytes[first + i] > largest) largest = bytes[first + i];
        }
        if (largest < 16) continue;
        size_t bx = (largest + 4096ull * 128 - 1) / (4096ull * 128);
        if (bx > 64) bx = 64;
        bs::l2_prefetch_kernel<<<dim3(static_cast<unsigned>(bx), static_cast<unsigned>(n)), 128, 0, static_cast<cudaStream_t>(stream)>>>(list);
        if (cudaGetLastError() != cudaSuccess) return BS_ERR_CUDA;
    }
    return BS_OK;
}

extern "C" int bs_popc_rate(int iters, double* wordops_per_s)
{
    if (iters <= 0 || wordops_per_s == nullptr) return BS_ERR_INVALID_ARG;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return BS_ERR_CUDA;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return BS_ERR_CUDA;
    int* sink = bs::status_device_ptr();
    if (!sink) return BS_ERR_CUDA;
    const int blocks = sms * 8, threads = 256;
    cudaEvent_t e0, e1;
    if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) return BS_ERR_CUDA;
    bs::popc_rate_kernel<<<blocks, threads>>>(iters / 4 + 1, 12345u, sink);   // warm-up
    cudaEventRecord(e0);
    bs::popc_rate_kernel<<<blocks, threads>>>(iters, 12345u, sink);
    cudaEventRecord(e1);
    cudaError_t err = cudaEventSynchronize(e1);
    float ms = 0.f;
    if (err == cudaSuccess) err = cudaEventElapsedTime(&ms, e0, e1);
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    if (err != cudaSuccess || cudaGetLastError() != cudaSuccess || ms <= 0.f) return BS_ERR_CUDA;
    const double ops = static_cast<double>(blocks) * threads * static_cast<double>(iters) * 32.0;
    *wordops_per_s = ops / (static_cast<double>(ms) * 1e-3);
    return BS_OK;
}

extern "C" int bs_check_status(void* stream)
{
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaStreamSynchronize(st) != cudaSuccess) { cudaGetLastError(); return BS_ERR_CUDA; }
    int h = 0;
    if (cudaMemcpyFromSymbol(&h, bs::g_status, sizeof(int)) != cudaSuccess) return BS_ERR_CUDA;
    if (h != 0) {
        int zero = 0;
        cudaMemcpyToSymbol(bs::g_status, &zero, sizeof(int));
        return BS_ERR_TIMEOUT;
    }
    return BS_OK;
}

extern "C" const char* bs_status_string(int status)
{
    switch (status) {
        case BS_OK: return "BS_OK";
        case BS_ERR_INVALID_ARG: return "BS_ERR_INVALID_ARG";
        case BS_ERR_UNSUPPORTED: return "BS_ERR_UNSUPPORTED";
        case BS_ERR_ALIGNMENT: return "BS_ERR_ALIGNMENT";
        case BS_ERR_CUDA: return "BS_ERR_CUDA";
        case BS_ERR_TIMEOUT: return "BS_ERR_TIMEOUT";
        default: return "BS_ERR_UNKNOWN";
    }
}
