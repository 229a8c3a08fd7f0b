// Entry points that are not kernels of their own: status strings, launch accounting and the
// host-buffer convenience call that chains copy-in, quantizer, linear layer and copy-out.
#include "tdq_common.cuh"

using namespace tdq;

extern "C" const char* tdq_status_string(tdq_status s) {
    switch (s) {
        case TDQ_OK: return "ok";
        case TDQ_ERR_INVALID_ARG: return "invalid argument";
        case TDQ_ERR_UNSUPPORTED: return "unsupported configuration";
        case TDQ_ERR_ALIGNMENT: return "misaligned pointer or stride";
        case TDQ_ERR_WORKSPACE: return "workspace missing or too small";
        case TDQ_ERR_CUDA: return "CUDA call failed";
        case TDQ_ERR_DEVICE_TIMEOUT: return "a bounded device-side wait ran out";
    }
    return "unknown status";
}

extern "C" uint64_t tdq_kernel_launch_count(void) { return g_launch_count.load(std::memory_order_relaxed); }

extern "C" tdq_status tdq_quant_linear_host(const void* x_host, tdq_dtype x_dtype, int64_t B, int64_t N, int64_t C,
                                            const tdq_act_params* p, const uint8_t* wcodes, const float* wscale,
                                            const float* bias, int64_t O, void* y_host, tdq_dtype y_dtype,
                                            void* x_dev, uint8_t* codes_dev, float* scale_dev, void* y_dev,
                                            void* workspace, size_t workspace_bytes, void* cuda_stream) {
    if (!x_host || !y_host || !x_dev || !codes_dev || !scale_dev || !y_dev || !p) return TDQ_ERR_INVALID_ARG;
    if (B < 0 || N < 0 || C <= 0 || O <= 0) return TDQ_ERR_INVALID_ARG;
    if (x_dtype != TDQ_F32 && x_dtype != TDQ_BF16) return TDQ_ERR_INVALID_ARG;
    if (y_dtype != TDQ_F32 && y_dtype != TDQ_BF16) return TDQ_ERR_INVALID_ARG;
    if (p->group_size <= 0) return TDQ_ERR_INVALID_ARG;
    const int64_t M = B * N;
    if (M == 0) return TDQ_OK;
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
    const size_t xbytes = (size_t)M * C * (x_dtype == TDQ_BF16 ? 2 : 4);
    const size_t ybytes = (size_t)M * O * (y_dtype == TDQ_BF16 ? 2 : 4);
    if (cudaMemcpyAsync(x_dev, x_host, xbytes, cudaMemcpyHostToDevice, stream) != cudaSuccess) return TDQ_ERR_CUDA;
    tdq_status st = tdq_quantize_act(x_dev, x_dtype, B, N, C, C, p, codes_dev, scale_dev, nullptr, cuda_stream);
    if (st != TDQ_OK) return st;
    const int64_t g = p->group_size;
    const int64_t I_pad = (C + g - 1) / g * g;
    st = tdq_w4a4_linear(codes_dev, scale_dev, wcodes, wscale, bias, M, I_pad, O, p->group_size, y_dev, y_dtype, O,
                         nullptr, workspace, workspace_bytes, cuda_stream);
    if (st != TDQ_OK) return st;
    if (cudaMemcpyAsync(y_host, y_dev, ybytes, cudaMemcpyDeviceToHost, stream) != cudaSuccess) return TDQ_ERR_CUDA;
    return TDQ_OK;
}
