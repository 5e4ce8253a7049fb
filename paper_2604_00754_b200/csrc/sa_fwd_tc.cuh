// Tensor-core (tcgen05 / TMEM) forward path: interface to the rest of the library.
#pragma once
#include "sa_common.cuh"

namespace sa {

// True when the bf16 tensor-core kernel can run this problem (shape, strides, alignment).
bool tc_forward_supported(const FwdArgs& a, int dtype);
cudaError_t launch_fwd_tc(const FwdArgs& a, cudaStream_t st);

}  // namespace sa
