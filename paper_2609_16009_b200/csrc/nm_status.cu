// Device status word, the driver entry point for tensor-map encoding, and nm_check_status().
#include <atomic>

#include <cudaTypedefs.h>

#include "nm_async.cuh"

namespace nm {

// Word 0: the status bits.  Word 1 (8 bytes further): the limit of a bounded wait in nanoseconds, read by mbar_wait
// through the same pointer the kernels already receive.
__device__ __align__(16) unsigned long long g_device_status[2] = {0ull, kWaitLimitNs};

unsigned *device_status_ptr()
{
    constexpr int kMaxDevices = 64;
    static std::atomic<unsigned *> cache[kMaxDevices] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    unsigned *p = cache[dev].load(std::memory_order_acquire);
    if (!p) {
        void *q = nullptr;
        if (cudaGetSymbolAddress(&q, g_device_status) != cudaSuccess) return nullptr;
        p = static_cast<unsigned *>(q);
        cache[dev].store(p, std::memory_order_release);          // two threads racing here store the same address
    }
    return p;
}

static EncodeTiledFn lookup_tensor_map_encoder()
{
    void *p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess && q == cudaDriverEntryPointSuccess)
        return reinterpret_cast<EncodeTiledFn>(p);
    return nullptr;
}

EncodeTiledFn tensor_map_encoder()
{
    static const EncodeTiledFn fn = lookup_tensor_map_encoder();   // initialised once, thread-safe
    return fn;
}

// One CTA that waits on an mbarrier nobody ever arrives at: the bounded wait runs out, raises the status word and
// the kernel returns normally.
__global__ void wait_probe_kernel(unsigned *status, unsigned long long *elapsed_ns)
{
    __shared__ __align__(8) unsigned long long bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(smem_u32(&bar), 1);
        mbar_init_fence();
    }
    __syncthreads();
    const unsigned long long t0 = global_timer_ns();
    const bool ok = mbar_wait(smem_u32(&bar), 0, &abort_flag, status);
    __syncthreads();
    // after the first expiry every later wait in the CTA gives up at once (the abort flag is up)
    const bool ok2 = mbar_wait(smem_u32(&bar), 0, &abort_flag, status);
    if (threadIdx.x == 0 && elapsed_ns) {
        elapsed_ns[0] = global_timer_ns() - t0;
        elapsed_ns[1] = (ok ? 1ull : 0ull) | (ok2 ? 2ull : 0ull);
    }
}

}  // namespace nm

extern "C" {
#pragma GCC visibility push(default)

int nm_check_status(nm_stream stream)
{
    unsigned *p = nm::device_status_ptr();
    if (!p) return NM_ERR_CUDA;
    unsigned v = 0;
    NM_CUDA_TRY(cudaStreamSynchronize((cudaStream_t)stream));
    NM_CUDA_TRY(cudaMemcpy(&v, p, sizeof v, cudaMemcpyDeviceToHost));
    if (v) {
        unsigned zero = 0;
        NM_CUDA_TRY(cudaMemcpy(p, &zero, sizeof zero, cudaMemcpyHostToDevice));
        return NM_ERR_TIMEOUT;
    }
    return NM_OK;
}

int nm_debug_wait_probe(unsigned long long limit_ns, unsigned long long *elapsed_ns, nm_stream stream)
{
    unsigned *p = nm::device_status_ptr();
    if (!p) return NM_ERR_CUDA;
    if (limit_ns < 1000ull || limit_ns > nm::kWaitLimitNs) return NM_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    // the limit word sits 8 bytes behind the status word; it goes back to its default right after the probe, in
    // stream order, so no other kernel on this stream ever sees the short limit
    const unsigned long long normal = nm::kWaitLimitNs;
    NM_CUDA_TRY(cudaMemcpyAsync(reinterpret_cast<char *>(p) + 8, &limit_ns, sizeof limit_ns, cudaMemcpyHostToDevice, s));
    nm::wait_probe_kernel<<<1, 64, 0, s>>>(p, elapsed_ns);
    cudaError_t e = cudaGetLastError();
    NM_CUDA_TRY(cudaMemcpyAsync(reinterpret_cast<char *>(p) + 8, &normal, sizeof normal, cudaMemcpyHostToDevice, s));
    if (e != cudaSuccess) return nm::record_cuda_error(e, "wait probe launch");
    return NM_OK;
}

#pragma GCC visibility pop
}
