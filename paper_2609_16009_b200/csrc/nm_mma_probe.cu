// Measurement aid: what one tcgen05.mma of a given shape costs on this part, operands in place.
//
// One CTA; one thread issues `reps` MMAs back to back (kind::f16, bf16 operands, K = 16) and one commit, and the
// clock is read before the first issue and after the commit has arrived.  The A operand comes from shared memory
// (K-major, 128-byte swizzle) or from TMEM; the B operand from shared memory, K-major or MN-major; the accumulator
// is one TMEM region or `n_acc` regions used in turn.  The operand bytes are whatever the (cleared) shared memory
// holds: only the time matters.  The kernels' tile shapes were chosen from these figures.
#include "nm_async.cuh"
#include "nm_tcgen05.cuh"

namespace nm {

namespace {

constexpr int kProbeSmem = 196608 + 1024;

__global__ void __launch_bounds__(128) mma_probe_kernel(int m, int n, int a_from_tmem, int b_mn_major, int reps, int n_acc, int a_step, int b_step,
                                                        unsigned long long *out, unsigned *status)
{
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t base = (raw_addr + 1023u) & ~1023u;
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;
    __shared__ __align__(8) unsigned long long bar_store;
    const uint32_t bar = smem_u32(&bar_store);
    const int tid = threadIdx.x, warp = tid >> 5;
    for (int i = tid; i < (kProbeSmem - 1024) / 16; i += blockDim.x)
        reinterpret_cast<uint4 *>(smem_raw + (base - raw_addr))[i] = make_uint4(0, 0, 0, 0);
    if (tid == 0) {
        s_abort = 0;
        mbar_init(bar, 1);
        mbar_init_fence();
    }
    if (warp == 1) tmem_alloc(&s_tmem_base, 512);
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = s_tmem_base;
    if (tid == 0) {
        const uint32_t idesc = instr_desc(m, n, false, b_mn_major != 0);
        // A: [m rows x 64 columns] blocks of 128-byte rows; B K-major: [n rows x 64 columns]; B MN-major: 64-column blocks
        // of [64 rows x 128 bytes] side by side (leading-dimension stride 8 KB), as the attention kernels lay them out
        const uint32_t a_addr = base, b_addr = base + 65536;
        const uint64_t a_desc0 = smem_desc(a_addr, 16, 1024);
        const uint64_t b_desc0 = b_mn_major ? smem_desc(b_addr, 8192, 1024) : smem_desc(b_addr, 16, 1024);
        // accumulators from column 0, n columns each; a TMEM A operand lives in the last 64 columns
        const uint32_t d0 = tmem, a_tmem = tmem + 448;
        // four operand positions and four accumulator choices, fixed before the clock starts: the loop body is four
        // bare MMA instructions
        uint64_t ad[4], bd[4];
        uint32_t dd[4], at[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            ad[j] = a_desc0 + (uint64_t)((j * a_step) >> 4);
            bd[j] = b_desc0 + (uint64_t)((j * b_step) >> 4);
            dd[j] = d0 + (uint32_t)((j % n_acc) * n);
            at[j] = a_tmem + 8 * j;
        }
        const int rounds = reps / 4;
        const long long t0 = clock64();
        if (a_from_tmem) {
#pragma unroll 1
            for (int i = 0; i < rounds; ++i) {
#pragma unroll
                for (int j = 0; j < 4; ++j) mma_ts(dd[j], at[j], bd[j], idesc, true);
            }
        } else {
#pragma unroll 1
            for (int i = 0; i < rounds; ++i) {
#pragma unroll
                for (int j = 0; j < 4; ++j) mma_ss(dd[j], ad[j], bd[j], idesc, true);
            }
        }
        const long long t_issued = clock64();
        mma_commit(bar);
        const bool ok = mbar_wait(bar, 0, &s_abort, status);
        const long long t1 = clock64();
        out[0] = (unsigned long long)(t1 - t0);
        out[1] = (unsigned long long)(t_issued - t0);
        out[2] = ok ? 1ull : 0ull;
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem, 512);
    }
}

}  // namespace

}  // namespace nm

extern "C" {
#pragma GCC visibility push(default)

int nm_debug_mma_probe(int m, int n, int a_from_tmem, int b_mn_major, int reps, int n_acc, int a_step_bytes, int b_step_bytes,
                       unsigned long long *out_clocks, nm_stream stream)
{
    using namespace nm;
    if ((m != 64 && m != 128) || n < 16 || n > 256 || n % 16 != 0 || reps < 1 || reps > 4096 || n_acc < 1 || n_acc * n > 448 || !out_clocks)
        return NM_ERR_INVALID_ARG;
    if (a_step_bytes < 0 || a_step_bytes > 8192 || b_step_bytes < 0 || b_step_bytes > 8192 || (a_step_bytes | b_step_bytes) % 16) return NM_ERR_INVALID_ARG;
    static std::atomic<unsigned long long> configured{0};
    cudaError_t e = ensure_dynamic_smem(mma_probe_kernel, kProbeSmem, configured);
    if (e != cudaSuccess) return record_cuda_error(e, "mma probe attribute");
    mma_probe_kernel<<<1, 128, kProbeSmem, (cudaStream_t)stream>>>(m, n, a_from_tmem, b_mn_major, reps, n_acc, a_step_bytes, b_step_bytes, out_clocks,
                                                                   device_status_ptr());
    e = cudaGetLastError();
    return e == cudaSuccess ? NM_OK : record_cuda_error(e, "mma probe launch");
}

#pragma GCC visibility pop
}
