// tdq_measure_mma_clocks: how fast the tensor core of this device runs the instruction the linear layer is
// built on, measured by the library itself (no counterpart in the paper).
//
// One CTA per SM issues a long run of tcgen05.mma instructions (M = 128, N = 128, K = 32, 8-bit operands) on
// operands that already sit in shared memory, with nothing else running: no copies, no promotion, no epilogue.
// The clocks per instruction that come out are the ceiling any kernel of this library can reach on the tensor
// pipe; the benchmark turns them into the dense 8-bit peak it quotes the linear layer against.
#include "tdq_tc.cuh"

namespace tdq {
namespace {

struct PeakRes {
    long long clocks;
    int32_t timed_out;
    int32_t pad;
};

template <bool I8>
__global__ void __launch_bounds__(128, 1) mma_rate_kernel(PeakRes* out, int n_mma) {
    extern __shared__ __align__(1024) uint8_t sm[];      // four K-steps of A, then four of B (zeros)
    __shared__ Ctrl c;
    __shared__ uint32_t status_word;                     // this kernel has no workspace: a wait that gives up notes it here
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int i = threadIdx.x; i < 2 * kChunk * kBlock / 4; i += blockDim.x) reinterpret_cast<uint32_t*>(sm)[i] = 0u;
    if (threadIdx.x == 0) {
        mbar_init(&c.tfull[0], 1);
        c.abort_flag = 0;
        status_word = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the zeros, before the tensor core reads them
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&c.tmem_base)),
                     "r"(kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = c.tmem_base;
    if (warp == 0) {
        const uint32_t lane0 = lane == 0 ? 1u : 0u;
        const uint32_t a0 = desc_lo(smem_u32(sm)), b0 = desc_lo(smem_u32(sm + kChunk * kBlock));
        const long long t0 = clock64();
#pragma unroll 1
        for (int i = 0; i < n_mma; i += kChunk)      // four K-steps chained into one accumulator, the accumulators in turn
            mma_issue4_if<I8>(lane0, tmem_base + (uint32_t)((i / kChunk) & (kSlots - 1)) * kBN, a0, b0, 0u);
        mma_commit_if(lane0, smem_u32(&c.tfull[0]));
        const bool ok = mbar_wait_warp(&c.tfull[0], 0u, &c, &status_word, 1u);
        if (lane == 0) {
            out[blockIdx.x].clocks = clock64() - t0;
            out[blockIdx.x].timed_out = ok ? 0 : 1;
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
}

}  // namespace
}  // namespace tdq

using namespace tdq;

extern "C" tdq_status tdq_measure_mma_clocks(int32_t integer_kind, int32_t n_mma, void* scratch, size_t scratch_bytes,
                                             double* clocks_per_mma, void* cuda_stream) {
    if (!scratch || !clocks_per_mma) return TDQ_ERR_INVALID_ARG;
    if (n_mma < kChunk || n_mma > (1 << 22) || n_mma % kChunk) return TDQ_ERR_INVALID_ARG;
    const int n_sm = current_device_sm_count();
    if (n_sm <= 0 || n_sm > 1024) return TDQ_ERR_CUDA;
    if (scratch_bytes < (size_t)n_sm * sizeof(PeakRes)) return TDQ_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(scratch) % 16) return TDQ_ERR_ALIGNMENT;
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
    auto kernel = integer_kind ? mma_rate_kernel<true> : mma_rate_kernel<false>;
    // more than half of the SM's shared memory, so that exactly one CTA runs on each (the kernel's own static
    // variables come on top of the dynamic part)
    constexpr int kDynSmem = 160 * 1024;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kDynSmem) != cudaSuccess) return TDQ_ERR_CUDA;
    kernel<<<n_sm, 128, kDynSmem, stream>>>(reinterpret_cast<PeakRes*>(scratch), n_mma);
    if (cudaGetLastError() != cudaSuccess) return TDQ_ERR_CUDA;
    g_launch_count.fetch_add(1, std::memory_order_relaxed);
    PeakRes host[1024];
    if (cudaMemcpyAsync(host, scratch, (size_t)n_sm * sizeof(PeakRes), cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
        cudaStreamSynchronize(stream) != cudaSuccess)
        return TDQ_ERR_CUDA;
    long long worst = 0;
    for (int i = 0; i < n_sm; ++i) {
        if (host[i].timed_out) return TDQ_ERR_DEVICE_TIMEOUT;
        if (host[i].clocks > worst) worst = host[i].clocks;
    }
    *clocks_per_mma = (double)worst / (double)n_mma;
    return TDQ_OK;
}
