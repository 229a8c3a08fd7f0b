// Shared host/device helpers of the tdq CUDA library (not used by the CPU oracle).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>
#include <utility>
#include <cmath>

#include "../../include/tdq.h"

namespace tdq {

// Numerical conventions of Supp. S4.8.
constexpr float kClipFloor = 1e-8f;   // every clip radius is at least this
constexpr float kStepFloor = 1e-8f;   // Delta = max(c / q_max, 1e-8)
constexpr float kStdEps = 1e-12f;     // sigma = Std + 1e-12
constexpr float kQmax = 7.0f;
// 1.5 * 2^23: adding it to |v| < 2^22 rounds v to the nearest integer, ties to even, and
// leaves that integer in the low mantissa bits as a two's complement offset.
constexpr float kRoundMagic = 12582912.0f;

extern std::atomic<uint64_t> g_launch_count;

// The linear layer with either source of its A operand.  fx == nullptr: activation codes and
// scales from memory (tdq_w4a4_linear).  Otherwise the activations themselves, quantized by the
// GEMM's own producer; xcodes and xscale are ignored.  pow2_steps != 0: tdq_w4a4_linear_pow2.
struct FusedSrc {
    const void* x;
    int64_t row_stride;   // elements
    bool bf16;
    float seven_tau;
    uint32_t flags;
};
tdq_status linear_impl(const FusedSrc* fx, const uint8_t* xcodes, const float* xscale, const uint8_t* wcodes,
                       const float* wscale, const float* bias, int64_t M, int64_t I_pad, int64_t O, int32_t group_size,
                       void* y, tdq_dtype y_dtype, int64_t y_row_stride, int32_t* acc_debug, void* workspace,
                       size_t workspace_bytes, void* cuda_stream, int pow2_steps);
// The shape, plan and workspace-size checks of tdq_w4a4_linear without its pointers: what a caller that chains
// several calls needs to know before it enqueues the first one (tdq_linear.cu).
tdq_status linear_check_shape(int64_t M, int64_t I_pad, int64_t O, int32_t group_size, size_t workspace_bytes);
// Argument checks of the quantizer and its fast-path conditions (tdq_quantize_act.cu).
tdq_status check_act_args(const void* x, tdq_dtype dt, int64_t B, int64_t N, int64_t C, int64_t stride,
                          const tdq_act_params* p);
bool act_fast_path_ok(const void* x, tdq_dtype dt, int64_t C, int64_t stride, const tdq_act_params* p);

// One warp waits, with the quantizer's ring-wait routine and the given cycle limit, on a barrier nobody arrives on
// (tdq_selftest_wait_timeout; tdq_quantize_act.cu).
tdq_status act_wait_selftest(long long limit_cycles, cudaStream_t stream);

// Bookkeeping kept per device (a process may drive several): the SM count of the current device, looked up once
// for each, and which devices a kernel's opt-in to large dynamic shared memory has been made on (the attribute
// belongs to the device's context).  Lock-free: a lost race only repeats an idempotent call.
constexpr int kMaxDevices = 64;
inline int current_device_sm_count(int* device = nullptr) {
    static std::atomic<int> cache[kMaxDevices];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return 0;
    if (device) *device = dev;
    int n = cache[dev].load(std::memory_order_relaxed);
    if (n == 0) {
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
        cache[dev].store(n, std::memory_order_relaxed);
    }
    return n;
}
// true once `done` has the device's bit; the caller sets the attribute when this returns false and then calls mark
inline bool device_marked(const std::atomic<uint64_t>& done, int dev) { return (done.load(std::memory_order_acquire) >> dev) & 1u; }
inline void mark_device(std::atomic<uint64_t>& done, int dev) { done.fetch_or(1ull << dev, std::memory_order_release); }

// Programmatic dependent launch.  The hot-path kernels are launched with the attribute that lets a grid start
// while its predecessor in the stream is still draining; each of them executes pdl_wait() in every thread before its
// first access to global memory (the wait returns when the preceding grids have completed and their writes are
// visible), so only block scheduling, shared-memory set-up and barrier initialisation overlap the predecessor's
// tail.  pdl_trigger() tells the scheduler that the next grid may be brought in.  Inside a captured graph the
// same launches become programmatic edges.  Kernels launched the ordinary way need neither call.
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
#endif
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

inline tdq_status cuda_status(cudaError_t e) { return e == cudaSuccess ? TDQ_OK : TDQ_ERR_CUDA; }

// Rank ceil(frac * g), 1-indexed, inside [1, g] (Supp. S2.2).  frac is a float, so a
// product within 1e-6 of an integer counts as that integer.
inline int32_t rank_of(float frac, int32_t g) {
    const double kd = (double)frac * (double)g;
    const double kr = std::floor(kd + 0.5);
    int64_t k = (std::fabs(kd - kr) < 1e-6) ? (int64_t)kr : (int64_t)std::ceil(kd);
    if (k < 1) k = 1;
    if (k > g) k = g;
    return (int32_t)k;
}

__device__ __forceinline__ float bf16_bits_to_float(uint32_t hi16) { return __uint_as_float(hi16 << 16); }

// DCRP, Eq. 12 with the floors of Supp. S4.8, in the binary32 order the paper writes:
// c first, then Delta = c / q_max.  No multiply-add may be fused here.
__device__ __forceinline__ void dcrp_project(float c_base, float sigma, float thr, float seven_tau,
                                             uint32_t flags, float& c, float& delta) {
    float cc = c_base;
    if (flags & TDQ_ENABLE_C1) cc = fminf(cc, __fmul_rn(seven_tau, sigma));
    if (flags & TDQ_ENABLE_C2) cc = fminf(cc, __fmul_rn(14.0f, thr));
    cc = fmaxf(cc, kClipFloor);
    c = cc;
    delta = fmaxf(__fdiv_rn(cc, kQmax), kStepFloor);
    if (flags & TDQ_POW2_STEP) {   // the power-of-two variant: drop the step's mantissa, keep c = 7 Delta
        delta = __uint_as_float(__float_as_uint(delta) & 0xff800000u);
        c = __fmul_rn(kQmax, delta);
    }
}

// One element of Alg. S1 steps 5 and 7 with a true IEEE division; returns the code.
__device__ __forceinline__ int quantize_ieee(float x, float c, float delta) {
    float xt = fminf(fmaxf(x, -c), c);
    float r = __fdiv_rn(xt, delta);
    int q = __float2int_rn(r);
    return max(-8, min(7, q));
}

}  // namespace tdq
