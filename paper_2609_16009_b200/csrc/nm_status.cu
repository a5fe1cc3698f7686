// Device status word, the driver entry point for tensor-map encoding, and nm_check_status().
#include <cudaTypedefs.h>

#include "nm_async.cuh"

namespace nm {

__device__ unsigned g_device_status = 0;

unsigned *device_status_ptr()
{
    constexpr int kMaxDevices = 64;
    static unsigned *cache[kMaxDevices] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    if (!cache[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_device_status) != cudaSuccess) return nullptr;
        cache[dev] = static_cast<unsigned *>(p);
    }
    return cache[dev];
}

EncodeTiledFn tensor_map_encoder()
{
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
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

#pragma GCC visibility pop
}
