// Host-visible interface of the operand pre-pass kernels.
#pragma once

#include <cstdint>
#include <cuda_runtime.h>

namespace mpg {

// out[r] = largest FP32 exponent field among the K elements of row r of X (rows x K, storage format of dtype)
cudaError_t launch_operand_exponents(int dtype, int rows, int K, const void *X, uint32_t *out, int num_sms,
                                     cudaStream_t stream);

// a kernel of one thread that does nothing (what a launch costs by itself)
cudaError_t launch_null(cudaStream_t stream);

}  // namespace mpg
