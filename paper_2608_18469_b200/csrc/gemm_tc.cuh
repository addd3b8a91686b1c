// Tensor-core GEMM path (tcgen05 + TMEM accumulators, operands staged by TMA) for bf16 models.
#pragma once
#include <cuda_runtime.h>

#include "kernels.cuh"

namespace erase {

struct TcPlan {
  int launches = 0;
};

// Decides whether the tensor-core kernel takes this GEMM (bf16 operands, aligned strides) and,
// if so, prepares everything the launch needs.  Returns false to leave it to the SIMT kernel.
bool tc_gemm_plan(const GemmArgs& g, TcPlan* plan);
cudaError_t tc_gemm_launch(const GemmArgs& g, const TcPlan& plan, cudaStream_t s);

}  // namespace erase
