// tdq_quant_linear_fused: the quantizer as the producer of the linear layer's A operand.
//
// The work is done by the linear layer's kernel (tdq_linear.cu) in its fused instantiation: at the
// start of each block of 128 token rows its promotion warps quantize the rows (the same per-group
// code as the stand-alone quantizer) and write operand bytes and scales into shared memory, where
// they stay for all of the block's column tiles.  This file holds the entry point's checks.
#include "tdq_common.cuh"

using namespace tdq;

extern "C" tdq_status tdq_quant_linear_fused(const void* x, tdq_dtype x_dtype, int64_t B, int64_t N, int64_t C,
                                             int64_t row_stride_elems, const tdq_act_params* p, const uint8_t* wcodes,
                                             const float* wscale, const float* bias, int64_t O, void* y,
                                             tdq_dtype y_dtype, int64_t y_row_stride, void* workspace,
                                             size_t workspace_bytes, void* cuda_stream) {
    tdq_status st = check_act_args(x, x_dtype, B, N, C, row_stride_elems, p);
    if (st != TDQ_OK) return st;
    // the producer is the fast path of the quantizer at its default rank
    if (p->group_size != 32 || C % 32 != 0 || !act_fast_path_ok(x, x_dtype, C, row_stride_elems, p))
        return TDQ_ERR_UNSUPPORTED;
    if ((p->flags & TDQ_ENABLE_C2) && rank_of(p->zr, 32) != 7) return TDQ_ERR_UNSUPPORTED;
    if (rank_of(p->base_percentile, 32) != 32) return TDQ_ERR_UNSUPPORTED;   // the producer takes the maximum as base radius
    FusedSrc fx;
    fx.x = x;
    fx.row_stride = row_stride_elems;
    fx.bf16 = x_dtype == TDQ_BF16;
    fx.seven_tau = 7.0f * p->tau;
    fx.flags = p->flags;
    return linear_impl(&fx, nullptr, nullptr, wcodes, wscale, bias, B * N, C, O, 32, y, y_dtype, y_row_stride, nullptr,
                       workspace, workspace_bytes, cuda_stream, 0);
}
