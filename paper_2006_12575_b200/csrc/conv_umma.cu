// tcgen05 implicit-GEMM convolution (placeholder until the tensor-core kernel lands).
#include "common.cuh"

namespace lamp {

bool umma_conv_fwd_supported(const ConvGeom &, const TView &, const TView &) { return false; }

lamp_status_t umma_conv_fwd(const ConvGeom &, const TView &, const bf16 *, const float *, const TView &, double *, int,
                            cudaStream_t)
{
    return LAMP_ERR_NOT_IMPLEMENTED;
}

size_t umma_dgrad_ws(const ConvGeom &g) { return align_up((size_t)27 * g.co * g.ci * sizeof(bf16), 256); }

lamp_status_t umma_transpose_weights(const bf16 *, bf16 *, int, int, int, cudaStream_t) { return LAMP_ERR_NOT_IMPLEMENTED; }

}  // namespace lamp
