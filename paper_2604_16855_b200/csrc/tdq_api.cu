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

namespace {

// Side streams and events of the host-buffer call, made once per process and device (the call is a
// convenience for callers who hold host data; it is the one entry point that creates CUDA objects).
constexpr int kHostChunks = 8;
struct HostPipe {
    cudaStream_t h2d = nullptr, d2h = nullptr;
    cudaEvent_t start = nullptr, done = nullptr, in[kHostChunks] = {}, out[kHostChunks] = {};
    bool ok = false;
};
HostPipe* host_pipe() {
    static HostPipe pipes[64];
    static std::atomic<int> guard{0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    HostPipe& p = pipes[dev];
    if (p.ok) return &p;
    while (guard.exchange(1, std::memory_order_acquire)) {}
    if (!p.ok) {
        bool good = cudaStreamCreateWithFlags(&p.h2d, cudaStreamNonBlocking) == cudaSuccess &&
                    cudaStreamCreateWithFlags(&p.d2h, cudaStreamNonBlocking) == cudaSuccess &&
                    cudaEventCreateWithFlags(&p.start, cudaEventDisableTiming) == cudaSuccess &&
                    cudaEventCreateWithFlags(&p.done, cudaEventDisableTiming) == cudaSuccess;
        for (int i = 0; i < kHostChunks && good; ++i)
            good = cudaEventCreateWithFlags(&p.in[i], cudaEventDisableTiming) == cudaSuccess &&
                   cudaEventCreateWithFlags(&p.out[i], cudaEventDisableTiming) == cudaSuccess;
        p.ok = good;
    }
    guard.store(0, std::memory_order_release);
    return p.ok ? &p : nullptr;
}

}  // namespace

// Rows go through in up to eight chunks so that the copy-out of one chunk (the long pole: y is eight
// times the size of x at cfg4) overlaps the copy-in and the kernels of the next; kernels run on the
// caller's stream, the copies on two side streams tied to it by events.
extern "C" tdq_status tdq_quant_linear_host(const void* x_host, tdq_dtype x_dtype, int64_t B, int64_t N, int64_t C,
                                            const tdq_act_params* p, const uint8_t* wcodes, const float* wscale,
                                            const float* bias, int64_t O, void* y_host, tdq_dtype y_dtype,
                                            void* x_dev, uint8_t* codes_dev, float* scale_dev, void* y_dev,
                                            void* workspace, size_t workspace_bytes, void* cuda_stream) {
    if (!x_host || !y_host || !x_dev || !codes_dev || !scale_dev || !y_dev || !p) return TDQ_ERR_INVALID_ARG;
    if (B < 0 || N < 0 || C <= 0 || O <= 0) return TDQ_ERR_INVALID_ARG;
    if (x_dtype != TDQ_F32 && x_dtype != TDQ_BF16) return TDQ_ERR_INVALID_ARG;
    if (y_dtype != TDQ_F32 && y_dtype != TDQ_BF16 && y_dtype != TDQ_F16) return TDQ_ERR_INVALID_ARG;
    // every check of the two calls that does not depend on a chunk's pointers is made here, before anything is
    // queued: a refusal must leave the streams untouched
    tdq_status chk = check_act_args(x_dev, x_dtype, B, N, C, C, p);
    if (chk != TDQ_OK) return chk;
    if (!wcodes || !wscale || !workspace) return wcodes && wscale ? TDQ_ERR_WORKSPACE : TDQ_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(wcodes) % 16 || reinterpret_cast<uintptr_t>(workspace) % 16 ||
        reinterpret_cast<uintptr_t>(codes_dev) % 16)
        return TDQ_ERR_ALIGNMENT;
    const int64_t M = B * N;
    if (M == 0) return TDQ_OK;
    {
        const int64_t g0 = p->group_size, Ip = (C + g0 - 1) / g0 * g0;
        int64_t rp = (M + kHostChunks - 1) / kHostChunks;
        rp = (rp + 127) / 128 * 128;
        if (((Ip / 2) * rp) % 16) return TDQ_ERR_ALIGNMENT;        // every chunk's codes must start 16-byte aligned
        chk = linear_check_shape(rp < M ? rp : M, Ip, O, p->group_size, workspace_bytes);
        if (chk != TDQ_OK) return chk;
    }
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
    HostPipe* hp = host_pipe();
    if (!hp) return TDQ_ERR_CUDA;
    const int64_t xe = x_dtype == TDQ_BF16 ? 2 : 4, ye = y_dtype == TDQ_F32 ? 4 : 2;
    const int64_t g = p->group_size;
    const int64_t K = (C + g - 1) / g, I_pad = K * g;
    int64_t rows_per = (M + kHostChunks - 1) / kHostChunks;
    rows_per = (rows_per + 127) / 128 * 128;
    if (cudaEventRecord(hp->start, stream) != cudaSuccess) return TDQ_ERR_CUDA;
    if (cudaStreamWaitEvent(hp->h2d, hp->start, 0) != cudaSuccess || cudaStreamWaitEvent(hp->d2h, hp->start, 0) != cudaSuccess)
        return TDQ_ERR_CUDA;
    int chunk = 0;
    for (int64_t m0 = 0; m0 < M; m0 += rows_per, ++chunk) {
        const int64_t rows = M - m0 < rows_per ? M - m0 : rows_per;
        const char* xh = reinterpret_cast<const char*>(x_host) + m0 * C * xe;
        char* xd = reinterpret_cast<char*>(x_dev) + m0 * C * xe;
        char* yd = reinterpret_cast<char*>(y_dev) + m0 * O * ye;
        if (cudaMemcpyAsync(xd, xh, (size_t)(rows * C * xe), cudaMemcpyHostToDevice, hp->h2d) != cudaSuccess ||
            cudaEventRecord(hp->in[chunk], hp->h2d) != cudaSuccess || cudaStreamWaitEvent(stream, hp->in[chunk], 0) != cudaSuccess)
            return TDQ_ERR_CUDA;
        tdq_status st = tdq_quantize_act(xd, x_dtype, 1, rows, C, C, p, codes_dev + m0 * (I_pad / 2), scale_dev + m0 * K, nullptr,
                                         cuda_stream);
        if (st != TDQ_OK) return st;
        st = tdq_w4a4_linear(codes_dev + m0 * (I_pad / 2), scale_dev + m0 * K, wcodes, wscale, bias, rows, I_pad, O,
                             p->group_size, yd, y_dtype, O, nullptr, workspace, workspace_bytes, cuda_stream);
        if (st != TDQ_OK) return st;
        if (cudaEventRecord(hp->out[chunk], stream) != cudaSuccess || cudaStreamWaitEvent(hp->d2h, hp->out[chunk], 0) != cudaSuccess ||
            cudaMemcpyAsync(reinterpret_cast<char*>(y_host) + m0 * O * ye, yd, (size_t)(rows * O * ye), cudaMemcpyDeviceToHost,
                            hp->d2h) != cudaSuccess)
            return TDQ_ERR_CUDA;
    }
    // the caller's stream finishes only after the last copy-out
    if (cudaEventRecord(hp->done, hp->d2h) != cudaSuccess || cudaStreamWaitEvent(stream, hp->done, 0) != cudaSuccess)
        return TDQ_ERR_CUDA;
    return TDQ_OK;
}
