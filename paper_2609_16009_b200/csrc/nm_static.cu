// nm_matmul_static: the narrow product for callers that cannot hand the library any scratch memory.
//
// The split-K partial sums and arrival counters live in a fixed array in the library's own device
// image instead of a caller-provided workspace, so this entry point never calls an allocator and
// needs no workspace argument.  The price is a fixed size limit and one shared scratch area per
// GPU (calls that overlap on the same GPU would overwrite each other's partial sums).
#include <mutex>

#include "nm_common.cuh"

// Lives in every GPU that loads the library, from load until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[NM_STATIC_SCRATCH_BYTES];

namespace {

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
void *g_scratch_addr[kMaxDevices] = {};      // device address of g_static_scratch, per device

// In host code `g_static_scratch` is only a handle for the runtime, not a device address: the
// address a kernel can use has to be asked for, once per device, with that device current.
int scratch_for_current_device(void **out, cudaStream_t stream)
{
    int dev = -1;
    NM_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return NM_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_addr[dev]) {
        void *p = nullptr;
        NM_CUDA_TRY(cudaGetSymbolAddress(&p, g_static_scratch));
        // The arrival counters at the front must start at zero.  The kernels put them back to zero
        // themselves, so this is needed once; the partial sums behind them are always written
        // before they are read and need no clearing.
        NM_CUDA_TRY(cudaMemsetAsync(p, 0, nm::kCounterBytes, stream));
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return NM_OK;
}

}  // namespace

extern "C" {
#pragma GCC visibility push(default)

int nm_matmul_static(const void *A, const void *B, void *C, int M, int N, int K,
                     nm_dtype dtype, nm_layout layout_B, nm_stream stream)
{
    cudaStream_t s = (cudaStream_t)stream;
    void *scratch = nullptr;
    int rc = scratch_for_current_device(&scratch, s);
    if (rc != NM_OK) return rc;
    rc = nm::matmul_enqueue(A, B, C, M, N, K, 1, K, 0, 0, N, 0, dtype, layout_B, scratch, NM_STATIC_SCRATCH_BYTES, s);
    // The only way the fixed scratch can be "missing or too small" is a problem beyond its limit.
    return rc == NM_ERR_WORKSPACE ? NM_ERR_TOO_LARGE : rc;
}

#pragma GCC visibility pop
}
