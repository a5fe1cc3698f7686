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

#ifdef NM_BOUNDS_CHECK
// The checked access macros on an address outside the span they are given (and inside the caller's buffer).
__global__ void bounds_selftest_kernel(unsigned *buf, size_t bytes, unsigned *out_loaded, unsigned *status)
{
    const Span first_half = make_span(buf, bytes / 2);
    unsigned *outside = buf + bytes / 8;                           // first word of the second half
    NM_ST(outside, 0xdeadbeefu, first_half, status);              // must not happen
    out_loaded[0] = NM_LD(outside, first_half, status);           // must yield 0
    NM_ST(buf, 0x600df00du, first_half, status);                  // inside: happens
    out_loaded[1] = NM_LD(buf, first_half, status);
}
#endif

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
        return (v & nm::kStatusOutOfBounds) ? NM_ERR_BOUNDS : NM_ERR_TIMEOUT;
    }
    return NM_OK;
}

/* 1 when this library is the debug build whose narrow-product kernels check every hand-indexed global access against its
 * operand's extent (NM_BOUNDS_CHECK), else 0. */
int nm_debug_bounds_checked(void)
{
#ifdef NM_BOUNDS_CHECK
    return 1;
#else
    return 0;
#endif
}

/* Debug build only: one thread stores to and loads from the first word of the SECOND half of `buf` through the checked
 * access macros while naming the FIRST half as the operand.  The word lies inside the caller's allocation, so nothing can
 * fault whether or not the check works; with the check the store is skipped (the word keeps its value), out_loaded[0]
 * receives 0 instead of the word, and nm_check_status reports NM_ERR_BOUNDS once.  NM_ERR_UNSUPPORTED in the normal build. */
int nm_debug_bounds_selftest(void *buf, size_t bytes, unsigned *out_loaded, nm_stream stream)
{
#ifdef NM_BOUNDS_CHECK
    if (!buf || bytes < 32 || (bytes & 7) || ((uintptr_t)buf & 3) || !out_loaded) return NM_ERR_INVALID_ARG;
    unsigned *p = nm::device_status_ptr();
    if (!p) return NM_ERR_CUDA;
    nm::bounds_selftest_kernel<<<1, 1, 0, (cudaStream_t)stream>>>(static_cast<unsigned *>(buf), bytes, out_loaded, p);
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? NM_OK : nm::record_cuda_error(e, "bounds self-test launch");
#else
    (void)buf; (void)bytes; (void)out_loaded; (void)stream;
    return NM_ERR_UNSUPPORTED;
#endif
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
