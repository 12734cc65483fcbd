// Host interface of the tensor-core (tcgen05 + TMA) variant of the skinny GEMM (gemm_tc.cu).
#pragma once
#include "gemm.cuh"

namespace csd {

bool tc_supported(int m, int N, int K, bool dual);
size_t tc_scratch_bytes(int m, int N, int K, bool dual);
int tc_ticket_count(int N);
csd_status launch_linear_tc(const LinearArgs& a, cudaStream_t st);

// 0 = automatic choice, 1 = CUDA-core kernel only, 2 = tensor-core kernel wherever it applies
void set_gemm_path(int path);
int gemm_path();

}  // namespace csd
