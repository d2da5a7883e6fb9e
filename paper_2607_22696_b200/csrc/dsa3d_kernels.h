// Internal launch interface between the C-ABI layer and the kernels.
#pragma once
#include <cuda_runtime.h>

#include "dsa3d_common.cuh"

namespace dsa3d {

cudaError_t launch_forward(const void* q, const void* k, const void* v, const float* offsets, void* out,
                           float* lse, const Problem& pr, bool bf16, cudaStream_t stream);

// acc_dk / acc_dv: fp32 accumulators [N, heads, d], zeroed by the caller.  For fp32 storage
// they are the dk / dv outputs themselves.
cudaError_t launch_backward(const void* q, const void* k, const void* v, const float* offsets,
                            const float* lse, const void* dout, void* dq, float* acc_dk, float* acc_dv,
                            float* doffsets, const Problem& pr, bool bf16, cudaStream_t stream);

// fp32 accumulators -> bf16 outputs (round to nearest even).
cudaError_t launch_convert_bf16(const float* acc, void* dst, long long count, cudaStream_t stream);

}  // namespace dsa3d
