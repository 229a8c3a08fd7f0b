// tdq_w4a4_linear: W4A4 linear layer on the 5th-generation tensor cores (Algorithm S1 step 10).
//
//   acc[m,o,k] = sum_{i in group k} q_x[m,i] q_w[o,i]      tcgen05.mma kind::i8, int32 in TMEM
//   y[m,o]     = s_o * sum_k Delta[m,k] * acc[m,o,k] + b_o  fp32 in registers
//
// The activation scale changes every g codes along the contraction axis, so an int32
// accumulator may only span one token-group.  Each group gets its own TMEM slot (a fresh
// accumulation; groups wider than 32 codes chain g/32 instructions into the same slot), is
// read back with tcgen05.ld, converted and multiplied by its Delta, and added to a float
// accumulator that lives in registers for the whole contraction.
//
// Operands.  Packed codes (16 bytes = 32 codes per row and K-step) are loaded with 128-bit
// loads and unpacked to int8 in shared memory.  A nibble is moved to the HIGH half of its
// byte, which is the two's complement byte 16 q: no sign extension is needed, the integer
// result is 256 acc (exactly; |256 acc| < 2^31 for g <= 4096) and the factor 1/256 is folded
// into Delta, an exact power-of-two scaling.  Even channels fill the first 16 bytes of a row
// and odd channels the second 16; both operands use the same order, so the sum is unchanged.
//
// Shared-memory operand layout: K-major, no swizzle.  A 32-byte row splits into two 16-byte
// chunks; 8 rows x 16 bytes form one contiguous 128-byte core matrix; the two K-chunks of an
// 8-row band are 128 bytes apart (leading byte offset), bands are 256 bytes apart (stride
// byte offset).
//
// Every wait on an mbarrier is bounded: after about a second the thread records a code in
// the workspace status word, the CTA stops waiting, releases its TMEM and returns.
#include "tdq_common.cuh"

namespace tdq {
namespace {

constexpr int kBM = 128;              // rows per CTA tile = TMEM lanes
constexpr int kRound = 4;             // K-steps (of 32 codes) staged per round
constexpr int kThreads = 128;
constexpr long long kTimeoutCycles = 2000000000LL;

struct LinArgs {
    const uint8_t* xcodes;
    const float* xscale;
    const uint8_t* wcodes;
    const float* wscale;
    const float* bias;
    int64_t M, O;
    int32_t row_bytes;      // I_pad / 2
    int32_t n_steps;        // I_pad / 32
    int32_t steps_per_grp;  // g / 32
    int32_t Kg;             // groups per token
    void* y;
    int64_t y_stride;
    int32_t* acc_debug;
    uint32_t* status;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}

__device__ __forceinline__ bool mbar_test(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}

// Bounded wait.  Returns false (after recording `code`) when the phase did not complete in time.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, uint32_t* status, uint32_t code) {
    if (mbar_test(bar, parity)) return true;
    const long long t0 = clock64();
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 64; ++i)
            if (mbar_test(bar, parity)) return true;
        if (clock64() - t0 > kTimeoutCycles) {
            atomicCAS(status, 0u, code);
            return false;
        }
    }
}

__device__ __forceinline__ uint64_t smem_desc_kmajor_noswizzle(uint32_t saddr) {
    // start address, leading byte offset 128, stride byte offset 256 (all >> 4), version 1
    return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)(128 >> 4) << 16) | ((uint64_t)(256 >> 4) << 32) |
           (1ull << 46);
}

__device__ __forceinline__ void mma_i8(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                       uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}

__device__ __forceinline__ void mma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
                 : "memory");
}

__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
          "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
          "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr)
        : "memory");
}

__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// 16 packed bytes (32 codes) -> two 16-byte chunks of bytes 16*q: even channels, odd channels.
__device__ __forceinline__ void unpack16(const uint4 p, uint4& even, uint4& odd) {
    even = make_uint4((p.x << 4) & 0xF0F0F0F0u, (p.y << 4) & 0xF0F0F0F0u, (p.z << 4) & 0xF0F0F0F0u,
                      (p.w << 4) & 0xF0F0F0F0u);
    odd = make_uint4(p.x & 0xF0F0F0F0u, p.y & 0xF0F0F0F0u, p.z & 0xF0F0F0F0u, p.w & 0xF0F0F0F0u);
}

// byte offset of row r, K-chunk 0 inside one K-step's operand block (see the layout note above)
__device__ __forceinline__ uint32_t row_off(int r) { return (uint32_t)((r >> 3) * 256 + (r & 7) * 16); }

template <int BN, bool YBF16>
__global__ void __launch_bounds__(kThreads) w4a4_linear_kernel(LinArgs a) {
    constexpr int kABytes = kBM * 32, kBBytes = BN * 32;
    constexpr uint32_t kCols = kRound * BN;        // TMEM columns: one slot of BN per group in flight
    constexpr uint32_t kIdesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) |
                                ((uint32_t)(kBM >> 4) << 24);   // S32 accum, signed 8-bit A and B, K-major
    __shared__ __align__(128) uint8_t sA[kRound * kABytes];
    __shared__ __align__(128) uint8_t sB[kRound * kBBytes];
    __shared__ __align__(8) uint64_t mma_bar;
    __shared__ uint32_t tmem_base_smem;
    __shared__ int aborted;

    const int t = threadIdx.x, warp = t >> 5;
    const int64_t m0 = (int64_t)blockIdx.x * kBM;
    const int64_t n0 = (int64_t)blockIdx.y * BN;
    const int64_t m = m0 + t;

    if (t == 0) {
        mbar_init(&mma_bar, 1);
        aborted = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_smem)),
                     "r"(kCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_smem;

    float yacc[BN];
#pragma unroll
    for (int j = 0; j < BN; ++j) yacc[j] = 0.0f;

    uint32_t phase = 0;
    for (int s0 = 0; s0 < a.n_steps; s0 += kRound) {
        const int nb = min(kRound, a.n_steps - s0);
        // ---- stage: unpack this round's K-steps of both operands into shared memory
        for (int b = 0; b < nb; ++b) {
            const int64_t col = (int64_t)(s0 + b) * 16;
            uint4 p = make_uint4(0, 0, 0, 0);
            if (m < a.M) p = __ldg(reinterpret_cast<const uint4*>(a.xcodes + m * a.row_bytes + col));
            uint4 ev, od;
            unpack16(p, ev, od);
            uint8_t* dst = sA + b * kABytes + row_off(t);
            *reinterpret_cast<uint4*>(dst) = ev;
            *reinterpret_cast<uint4*>(dst + 128) = od;
#pragma unroll
            for (int j = t; j < BN; j += kThreads) {
                const int64_t n = n0 + j;
                uint4 pw = make_uint4(0, 0, 0, 0);
                if (n < a.O) pw = __ldg(reinterpret_cast<const uint4*>(a.wcodes + n * a.row_bytes + col));
                unpack16(pw, ev, od);
                uint8_t* dw = sB + b * kBBytes + row_off(j);
                *reinterpret_cast<uint4*>(dw) = ev;
                *reinterpret_cast<uint4*>(dw + 128) = od;
            }
        }
        fence_async_smem();
        __syncthreads();
        // ---- one thread issues the round's MMAs
        if (t == 0) {
            tc_fence_after();
            for (int b = 0; b < nb; ++b) {
                const int step = s0 + b;
                const int grp = step / a.steps_per_grp;
                const uint32_t first = (step % a.steps_per_grp) == 0 ? 0u : 1u;
                mma_i8(tmem_base + (uint32_t)(grp % kRound) * BN, smem_desc_kmajor_noswizzle(smem_u32(sA + b * kABytes)),
                       smem_desc_kmajor_noswizzle(smem_u32(sB + b * kBBytes)), kIdesc, first);
            }
            mma_commit(&mma_bar);
        }
        // ---- wait for the tensor core, then promote every group that ended in this round
        if (!aborted && !mbar_wait(&mma_bar, phase, a.status, 1u | ((uint32_t)blockIdx.x << 8))) aborted = 1;
        phase ^= 1;
        tc_fence_after();
        for (int b = 0; b < nb; ++b) {
            const int step = s0 + b;
            if ((step % a.steps_per_grp) != a.steps_per_grp - 1) continue;
            const int grp = step / a.steps_per_grp;
            const float d256 = (m < a.M) ? a.xscale[m * a.Kg + grp] * (1.0f / 256.0f) : 0.0f;
            const uint32_t taddr = tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)(grp % kRound) * BN;
#pragma unroll
            for (int c = 0; c < BN; c += 32) {
                uint32_t v[32];
                tmem_ld32(taddr + c, v);
                tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 32; ++j) yacc[c + j] = fmaf(d256, (float)(int32_t)v[j], yacc[c + j]);
                if (a.acc_debug && m < a.M) {
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        if (n0 + c + j < a.O) a.acc_debug[(m * a.O + n0 + c + j) * a.Kg + grp] = ((int32_t)v[j]) >> 8;
                }
            }
        }
        tc_fence_before();
        __syncthreads();
    }

    // ---- epilogue: y = s_o * sum + bias
    if (m < a.M) {
#pragma unroll
        for (int j = 0; j < BN; ++j) {
            const int64_t n = n0 + j;
            if (n < a.O) {
                const float b = a.bias ? a.bias[n] : 0.0f;
                const float v = __fmaf_rn(a.wscale[n], yacc[j], b);
                if (YBF16)
                    reinterpret_cast<__nv_bfloat16*>(a.y)[m * a.y_stride + n] = __float2bfloat16_rn(v);
                else
                    reinterpret_cast<float*>(a.y)[m * a.y_stride + n] = v;
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kCols) : "memory");
}

}  // namespace
}  // namespace tdq

using namespace tdq;

extern "C" size_t tdq_linear_workspace_bytes(int64_t, int64_t, int64_t, int32_t) { return 256; }

extern "C" tdq_status tdq_w4a4_linear(const uint8_t* xcodes, const float* xscale, const uint8_t* wcodes,
                                      const float* wscale, const float* bias, int64_t M, int64_t I_pad, int64_t O,
                                      int32_t group_size, void* y, tdq_dtype y_dtype, int64_t y_row_stride,
                                      int32_t* acc_debug, void* workspace, size_t workspace_bytes,
                                      void* cuda_stream) {
    if (!xcodes || !xscale || !wcodes || !wscale || !y) return TDQ_ERR_INVALID_ARG;
    if (M < 0 || O <= 0 || I_pad <= 0 || y_row_stride < O) return TDQ_ERR_INVALID_ARG;
    if (y_dtype != TDQ_F32 && y_dtype != TDQ_BF16) return TDQ_ERR_INVALID_ARG;
    if (group_size <= 0 || I_pad % group_size) return TDQ_ERR_INVALID_ARG;
    if (group_size % 32 || group_size > 4096) return TDQ_ERR_UNSUPPORTED;
    if (!workspace || workspace_bytes < tdq_linear_workspace_bytes(M, I_pad, O, group_size)) return TDQ_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(xcodes) % 16 || reinterpret_cast<uintptr_t>(wcodes) % 16 ||
        reinterpret_cast<uintptr_t>(workspace) % 16)
        return TDQ_ERR_ALIGNMENT;
    if (I_pad / 2 > INT32_MAX) return TDQ_ERR_INVALID_ARG;
    if (M == 0) return TDQ_OK;
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
    if (cudaMemsetAsync(workspace, 0, 16, stream) != cudaSuccess) return TDQ_ERR_CUDA;

    LinArgs a;
    a.xcodes = xcodes; a.xscale = xscale; a.wcodes = wcodes; a.wscale = wscale; a.bias = bias;
    a.M = M; a.O = O;
    a.row_bytes = (int32_t)(I_pad / 2);
    a.n_steps = (int32_t)(I_pad / 32);
    a.steps_per_grp = group_size / 32;
    a.Kg = (int32_t)(I_pad / group_size);
    a.y = y; a.y_stride = y_row_stride; a.acc_debug = acc_debug;
    a.status = reinterpret_cast<uint32_t*>(workspace);

    const int64_t mt = (M + kBM - 1) / kBM;
    const bool bf = (y_dtype == TDQ_BF16);
    if (O <= 64) {
        dim3 grid((unsigned)mt, (unsigned)((O + 63) / 64));
        if (bf) w4a4_linear_kernel<64, true><<<grid, kThreads, 0, stream>>>(a);
        else w4a4_linear_kernel<64, false><<<grid, kThreads, 0, stream>>>(a);
    } else {
        dim3 grid((unsigned)mt, (unsigned)((O + 127) / 128));
        if (bf) w4a4_linear_kernel<128, true><<<grid, kThreads, 0, stream>>>(a);
        else w4a4_linear_kernel<128, false><<<grid, kThreads, 0, stream>>>(a);
    }
    if (cudaGetLastError() != cudaSuccess) return TDQ_ERR_CUDA;
    g_launch_count.fetch_add(1, std::memory_order_relaxed);
    return TDQ_OK;
}

extern "C" tdq_status tdq_workspace_status(const void* workspace, void* cuda_stream, uint32_t* detail) {
    if (!workspace) return TDQ_ERR_INVALID_ARG;
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
    uint32_t word = 0;
    if (cudaMemcpyAsync(&word, workspace, sizeof word, cudaMemcpyDeviceToHost, stream) != cudaSuccess) return TDQ_ERR_CUDA;
    if (cudaStreamSynchronize(stream) != cudaSuccess) return TDQ_ERR_CUDA;
    if (detail) *detail = word;
    return word == 0 ? TDQ_OK : TDQ_ERR_DEVICE_TIMEOUT;
}
