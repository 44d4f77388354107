// Launchers of the LoPA-approximation kernels (see cast_kernels.cu).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace sffn {

cudaError_t launch_lopa_m_step(const float* W, const float* P, int H, int D, int32_t* g_idx, int8_t* g_sign,
                               double* row_energy, float* row_best, cudaStream_t s);
cudaError_t launch_lopa_residual(const float* W, const int32_t* g_idx, const int8_t* g_sign, int H, int D, float* A,
                                 cudaStream_t s);

}  // namespace sffn
