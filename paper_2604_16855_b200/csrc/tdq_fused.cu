// tdq_quant_linear_fused: the quantizer as the producer of the linear layer's A operand.
#include "tdq_common.cuh"

using namespace tdq;

extern "C" tdq_status tdq_quant_linear_fused(const void*, tdq_dtype, int64_t, int64_t, int64_t, int64_t,
                                             const tdq_act_params*, const uint8_t*, const float*, const float*,
                                             int64_t, void*, tdq_dtype, int64_t, void*, size_t, void*) {
    return TDQ_ERR_UNSUPPORTED;
}
