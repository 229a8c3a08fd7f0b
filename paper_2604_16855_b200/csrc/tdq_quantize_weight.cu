// tdq_quantize_weight: static per-output-channel symmetric 4-bit weight quantizer (Eq. 4).
// One CTA per output channel: absmax over the row, s_o = max(absmax / 7, 1e-8), then
// Q = clip(rint(W / s_o), -8, 7) with an IEEE division, two codes per byte.  Runs once
// per layer, so it is written for clarity, not for bandwidth.
#include "tdq_common.cuh"

namespace tdq {
namespace {

constexpr int kWThreads = 256;

template <bool BF16>
__global__ void __launch_bounds__(kWThreads) weight_quant_kernel(const void* w, int64_t I, int64_t I_pad,
                                                                  uint8_t* wcodes, float* wscale) {
    __shared__ uint32_t warp_max[kWThreads / 32];
    __shared__ float s_shared;
    const int64_t o = blockIdx.x;
    const int64_t base = o * I;
    uint32_t kmax = 0;   // bit pattern of the largest |w|
    for (int64_t i = threadIdx.x; i < I; i += kWThreads) {
        float v = BF16 ? bf16_bits_to_float(reinterpret_cast<const uint16_t*>(w)[base + i])
                       : reinterpret_cast<const float*>(w)[base + i];
        kmax = max(kmax, __float_as_uint(fabsf(v)));
    }
    kmax = __reduce_max_sync(0xffffffffu, kmax);
    if ((threadIdx.x & 31) == 0) warp_max[threadIdx.x >> 5] = kmax;
    __syncthreads();
    if (threadIdx.x == 0) {
        uint32_t m = 0;
        for (int i = 0; i < kWThreads / 32; ++i) m = max(m, warp_max[i]);
        float s = fmaxf(__fdiv_rn(__uint_as_float(m), kQmax), kStepFloor);
        s_shared = s;
        wscale[o] = s;
    }
    __syncthreads();
    const float s = s_shared;
    for (int64_t j = threadIdx.x; j < I_pad / 2; j += kWThreads) {
        int q[2];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            int64_t i = 2 * j + h;
            float v = 0.0f;
            if (i < I)
                v = BF16 ? bf16_bits_to_float(reinterpret_cast<const uint16_t*>(w)[base + i])
                         : reinterpret_cast<const float*>(w)[base + i];
            int qi = __float2int_rn(__fdiv_rn(v, s));
            q[h] = max(-8, min(7, qi));
        }
        wcodes[o * (I_pad / 2) + j] = (uint8_t)((q[0] & 0xF) | ((q[1] & 0xF) << 4));
    }
}

// The affine output correction folded into the layer's constants: a (s Sigma + bias) + b = (a s) Sigma + (a bias + b).
__global__ void fold_affine_kernel(const float* wscale, const float* bias, const float* mul, const float* add, int64_t O,
                                   float* wscale_out, float* bias_out) {
    const int64_t o = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (o >= O) return;
    const float a = mul[o];
    wscale_out[o] = __fmul_rn(a, wscale[o]);
    const float ab = bias ? __fmul_rn(a, bias[o]) : 0.0f;
    bias_out[o] = add ? __fadd_rn(ab, add[o]) : ab;
}

}  // namespace
}  // namespace tdq

using namespace tdq;

extern "C" tdq_status tdq_quantize_weight(const void* w, tdq_dtype w_dtype, int64_t O, int64_t I, int32_t pad_to,
                                          uint8_t* wcodes, float* wscale, void* cuda_stream) {
    if (!w || !wcodes || !wscale) return TDQ_ERR_INVALID_ARG;
    if (w_dtype != TDQ_F32 && w_dtype != TDQ_BF16) return TDQ_ERR_INVALID_ARG;
    if (O < 0 || I <= 0 || pad_to < 2 || (pad_to & 1) || O > INT32_MAX) return TDQ_ERR_INVALID_ARG;
    if (O == 0) return TDQ_OK;
    const int64_t I_pad = (I + pad_to - 1) / pad_to * pad_to;
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
    if (w_dtype == TDQ_BF16)
        weight_quant_kernel<true><<<(unsigned)O, kWThreads, 0, stream>>>(w, I, I_pad, wcodes, wscale);
    else
        weight_quant_kernel<false><<<(unsigned)O, kWThreads, 0, stream>>>(w, I, I_pad, wcodes, wscale);
    if (cudaGetLastError() != cudaSuccess) return TDQ_ERR_CUDA;
    g_launch_count.fetch_add(1, std::memory_order_relaxed);
    return TDQ_OK;
}

extern "C" tdq_status tdq_fold_output_affine(const float* wscale, const float* bias, const float* out_mul, const float* out_add,
                                             int64_t O, float* wscale_out, float* bias_out, void* cuda_stream) {
    if (!wscale || !out_mul || !wscale_out || !bias_out) return TDQ_ERR_INVALID_ARG;
    if (O < 0 || O > INT32_MAX) return TDQ_ERR_INVALID_ARG;
    if (O == 0) return TDQ_OK;
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
    fold_affine_kernel<<<(unsigned)((O + 255) / 256), 256, 0, stream>>>(wscale, bias, out_mul, out_add, O, wscale_out, bias_out);
    if (cudaGetLastError() != cudaSuccess) return TDQ_ERR_CUDA;
    g_launch_count.fetch_add(1, std::memory_order_relaxed);
    return TDQ_OK;
}
