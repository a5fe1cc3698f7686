// Read-only streaming probe: what this GPU delivers when a kernel does nothing but read memory once, the way
// the narrow products read their weights.  The roofline's denominator is a measured COPY (read + write); a
// read-only stream runs a little faster, and this puts a number on it beside the products' own.
#include "nm_common.cuh"

namespace nm {

namespace {

// Each thread reads 16 bytes per step with the same streaming load as the kernels, eight loads in flight,
// and folds them into one word; one word per CTA is written so that the loads cannot be dropped.
__global__ void __launch_bounds__(256) stream_read_kernel(const uint4 *__restrict__ src, long n16, unsigned *__restrict__ sink)
{
    const long stride = (long)gridDim.x * blockDim.x;
    long i = (long)blockIdx.x * blockDim.x + threadIdx.x;
    unsigned acc = 0;
    for (; i + 7 * stride < n16; i += 8 * stride) {
        uint4 v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) v[u] = ld_stream16(src + i + u * stride);
#pragma unroll
        for (int u = 0; u < 8; ++u) acc ^= v[u].x ^ v[u].y ^ v[u].z ^ v[u].w;
    }
    for (; i < n16; i += stride) {
        const uint4 v = ld_stream16(src + i);
        acc ^= v.x ^ v.y ^ v.z ^ v.w;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc ^= __shfl_xor_sync(0xffffffffu, acc, o);
    if ((threadIdx.x & 31) == 0 && acc == 0x9e3779b9u) atomicXor(sink, acc);       // practically never: keeps the loads alive
}

}  // namespace

}  // namespace nm

extern "C" {
#pragma GCC visibility push(default)

int nm_debug_stream_read(const void *src, size_t bytes, void *sink4, int ctas_per_sm, nm_stream stream)
{
    if (!src || !sink4 || bytes < 16 || ((uintptr_t)src & 15u) || ((uintptr_t)sink4 & 3u)) return NM_ERR_INVALID_ARG;
    if (ctas_per_sm < 1 || ctas_per_sm > 8) return NM_ERR_INVALID_ARG;
    int dev = 0, sms = 0;
    NM_CUDA_TRY(cudaGetDevice(&dev));
    NM_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    nm::stream_read_kernel<<<sms * ctas_per_sm, 256, 0, (cudaStream_t)stream>>>(static_cast<const uint4 *>(src), (long)(bytes / 16),
                                                                                static_cast<unsigned *>(sink4));
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? NM_OK : nm::record_cuda_error(e, "stream probe launch");
}

#pragma GCC visibility pop
}
