// Host-side helpers shared by the translation units that implement entry points of the C ABI.
#pragma once
#include <cuda_runtime.h>

#include "../../include/pivot.h"

namespace pivot {

// Argument checks common to every entry point (pointers, operand types, alignment, supported
// shapes); returns PIVOT_OK or the error code the entry point must return.
int check_operands(const pivot_tensor* q, const float* w, const pivot_tensor* kc, int H, int d, int c, int k,
                   int mode, const void* out);

// PIVOT_OK for cudaSuccess; otherwise remembers the code for pivot_last_cuda_error and returns
// PIVOT_ERR_CUDA.
int record_cuda(cudaError_t e);

}  // namespace pivot
