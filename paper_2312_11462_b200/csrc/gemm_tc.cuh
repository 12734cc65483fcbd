// Host interface of the tensor-core (tcgen05 + TMA) variant of the skinny GEMM (gemm_tc.cu).
#pragma once
#include "gemm.cuh"

namespace csd {

bool tc_supported(int m, int N, int K, bool dual);
size_t tc_scratch_bytes(int m, int N, int K, bool dual);
int tc_ticket_count(int N);
csd_status launch_linear_tc(const LinearArgs& a, cudaStream_t st);

// Several dependent GEMMs in one persistent kernel (gemm_chain.cu).  ops[j+1].xs must be what
// ops[j] writes as out_xs; ops[0].xs must be ready; all share m, ops[0].partial (chain_scratch_bytes)
// and ops[0].tickets (room for the tiles of all of them).  done_dev: 4 zero-initialised counters.
constexpr int CHAIN_OPS_MAX = 4;
size_t chain_scratch_bytes(int m);
csd_status launch_linear_chain(const LinearArgs* ops, int n_ops, unsigned* done_dev, unsigned* epoch_host,
                               cudaStream_t st);

// 0 = automatic choice, 1 = CUDA-core kernel only, 2 = tensor-core kernel wherever it applies
void set_gemm_path(int path);
int gemm_path();

}  // namespace csd
