// Tensor-core (tcgen05 / TMEM) backward path: interface to the rest of the library.
#pragma once
#include "sa_common.cuh"

namespace sa {

// True when the bf16 tensor-core kernels can run this backward problem.
bool tc_backward_supported(const BwdArgs& a, int dtype);
// dq, dk, dv of every branch; expects a.delta to be filled (bwd_delta_kernel) already.
cudaError_t launch_bwd_tc(const BwdArgs& a, cudaStream_t st);

}  // namespace sa
